"""Pins for the CPU checker's update rules (Eq. sgd, Eq. adam) and the 8-bit step built
around them (Section I / IV-B: 8-bit -> 32-bit, update, quantize back).  No CUDA here.

Hand-computed cases use dyadic numbers, so the expected values below are exact decimal
literals, not a re-typed formula.  torch.optim is the library special case the update
reduces to when the states are exact fp32.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2412_01195_b200 import synth

F = np.float32
BC = oracle.FLAG_BIAS_CORRECTION
DW = oracle.FLAG_DECOUPLED_WD


def arr(*v):
    return np.array(v, np.float32)


# ------------------------------------------------------------------------------------------
# Eq. sgd
# ------------------------------------------------------------------------------------------
def test_sgd_hand_computed():
    """beta = 1/2, lr = 1/4: m_0 = g_0; m_t = m_{t-1}/2 + g_t; w_t = w_{t-1} - m_t/4."""
    w, m = arr(1.0, -2.0, 0.5), arr(0, 0, 0)
    oracle.sgd_update_fp32(w, arr(0.5, 1.0, -0.25), m, 0.25, 0.5, 0.0)
    assert m.tolist() == [0.5, 1.0, -0.25]                   # m_0 = g_0
    assert w.tolist() == [0.875, -2.25, 0.5625]
    oracle.sgd_update_fp32(w, arr(0.25, -1.0, 0.0), m, 0.25, 0.5, 0.0)
    assert m.tolist() == [0.5, -0.5, -0.125]
    assert w.tolist() == [0.75, -2.125, 0.59375]


def test_sgd_weight_decay_hand_computed():
    """wd = 1/2 enters the gradient before the momentum: g' = g + w/2."""
    w, m = arr(2.0, -4.0), arr(1.0, 0.0)
    oracle.sgd_update_fp32(w, arr(1.0, 0.0), m, 0.5, 0.5, 0.5)
    assert m.tolist() == [2.5, -2.0]                          # 0.5*1 + (1 + 1), 0 + (0 - 2)
    assert w.tolist() == [0.75, -3.0]


@pytest.mark.parametrize("wd", [0.0, 1e-4])
def test_sgd_matches_torch_optim(wd, paper_facts):
    n, steps, lr, beta = 4096, 100, 0.1, paper_facts["sgd_momentum"]
    w0 = synth.normal(n, 0.05, 21)
    p = torch.nn.Parameter(w0.clone())
    opt = torch.optim.SGD([p], lr=lr, momentum=beta, weight_decay=wd, dampening=0.0)
    w, m = w0.numpy().copy(), np.zeros(n, F)
    for t in range(steps):
        g = synth.student_t(n, 3, 1e-3, 2100 + t)
        p.grad = g.clone()
        opt.step()
        oracle.sgd_update_fp32(w, g.numpy(), m, lr, beta, wd)
    ref = p.detach().numpy()
    assert np.max(np.abs(w - ref)) <= 2e-6 * np.max(np.abs(ref))
    buf = opt.state[p]["momentum_buffer"].numpy()
    assert np.max(np.abs(m - buf)) <= 2e-6 * np.max(np.abs(buf))


# ------------------------------------------------------------------------------------------
# Eq. adam
# ------------------------------------------------------------------------------------------
def test_adam_literal_equation_hand_computed():
    """No bias correction, eps = 0, beta1 = 1/2, beta2 = 3/4: after one step from zero state
    m = g/2, r = g^2/4, sqrt(r) = |g|/2, so w moves by exactly lr * sign(g)."""
    w, m, r = arr(1.0, 1.0, -3.0), arr(0, 0, 0), arr(0, 0, 0)
    oracle.adam_update_fp32(w, arr(0.5, -4.0, 0.125), m, r, 0.25, 0.5, 0.75, 0.0, 0.0, 1, flags=0)
    assert m.tolist() == [0.25, -2.0, 0.0625]
    assert r.tolist() == [0.0625, 4.0, 0.00390625]
    assert w.tolist() == [0.75, 1.25, -3.25]
    # second step, same gradients: m = 3g/4, r = 7g^2/16 -> not dyadic, check to rounding
    oracle.adam_update_fp32(w, arr(0.5, -4.0, 0.125), m, r, 0.25, 0.5, 0.75, 0.0, 0.0, 2, flags=0)
    assert m.tolist() == [0.375, -3.0, 0.09375]
    assert r.tolist() == [0.109375, 7.0, 0.0068359375]
    step = 0.25 * 0.75 / np.sqrt(7.0 / 16.0)
    assert np.allclose(w, [0.75 - step, 1.25 + step, -3.25 - step], rtol=3e-7)


def test_adam_bias_correction_hand_computed():
    """t = 1: m/(1-beta1) = g and r/(1-beta2) = g^2, so w_1 = w_0 - lr * g/(|g| + eps)."""
    w, m, r = arr(1.0, 1.0), arr(0, 0), arr(0, 0)
    oracle.adam_update_fp32(w, arr(2.0, -0.5), m, r, 0.5, 0.5, 0.75, 2.0, 0.0, 1, flags=BC)
    assert m.tolist() == [1.0, -0.25] and r.tolist() == [1.0, 0.0625]
    assert w[0] == 0.75 and w[1] == F(1.1)   # 1 - 0.5*2/(2+2), 1 + 0.5*0.5/(0.5+2) = 1.1 (rounded)
    # t = 2, betas 1/2 and 1/2: bc = 3/4 for both
    w, m, r = arr(0.0), arr(3.0), arr(3.0)
    oracle.adam_update_fp32(w, arr(0.0), m, r, 1.0, 0.5, 0.5, 0.0, 0.0, 2, flags=BC)
    assert m.tolist() == [1.5] and r.tolist() == [1.5]
    assert np.allclose(w, [-(1.5 / 0.75) / np.sqrt(1.5 / 0.75)], rtol=2e-7)


def test_adam_weight_decay_modes_hand_computed():
    # decoupled: w <- w (1 - lr wd) before the step; states see the raw gradient
    w, m, r = arr(4.0), arr(0.0), arr(0.0)
    oracle.adam_update_fp32(w, arr(1.0), m, r, 0.5, 0.5, 0.75, 0.0, 0.25, 1, flags=DW)
    assert m.tolist() == [0.5] and r.tolist() == [0.25]
    assert w.tolist() == [4.0 * 0.875 - 0.5]
    # coupled: g <- g + wd w = 2; m = 1, r = 1
    w, m, r = arr(4.0), arr(0.0), arr(0.0)
    oracle.adam_update_fp32(w, arr(1.0), m, r, 0.5, 0.5, 0.75, 0.0, 0.25, 1, flags=0)
    assert m.tolist() == [1.0] and r.tolist() == [1.0]
    assert w.tolist() == [3.5]


@pytest.mark.parametrize("decoupled", [True, False])
def test_adam_matches_torch_optim(decoupled, paper_facts):
    # betas as the binary32 numbers the C interface receives, so that torch (which forms
    # 1 - beta in binary64) and the checker (binary32) use the same coefficients
    n, steps, lr, b1, b2, eps = 4096, 100, 1e-3, float(F(0.9)), float(F(0.999)), 1e-8
    wd = paper_facts["adamw_weight_decay"]
    w0 = synth.normal(n, 0.02, 31)
    p = torch.nn.Parameter(w0.clone())
    cls = torch.optim.AdamW if decoupled else torch.optim.Adam
    opt = cls([p], lr=lr, betas=(b1, b2), eps=eps, weight_decay=wd)
    w, m, r = w0.numpy().copy(), np.zeros(n, F), np.zeros(n, F)
    flags = BC | (DW if decoupled else 0)
    for t in range(1, steps + 1):
        g = synth.normal(n, 1e-3, 3100 + t)
        p.grad = g.clone()
        opt.step()
        oracle.adam_update_fp32(w, g.numpy(), m, r, lr, b1, b2, eps, wd, t, flags)
    ref = p.detach().numpy()
    assert np.max(np.abs(w - ref)) <= 3e-6 * np.max(np.abs(ref))
    ea, es = opt.state[p]["exp_avg"].numpy(), opt.state[p]["exp_avg_sq"].numpy()
    assert np.max(np.abs(m - ea)) <= 3e-6 * np.max(np.abs(ea))
    assert np.max(np.abs(r - es)) <= 3e-6 * np.max(np.abs(es))


# ------------------------------------------------------------------------------------------
# the 8-bit step
# ------------------------------------------------------------------------------------------
def test_8bit_sgd_with_exactly_representable_states():
    """States that sit on code-book values survive the 8-bit storage exactly, so the 8-bit step
    must reproduce the hand-computed fp32 trajectory.  Block of 2: m = [max, 0] quantizes to
    codes [255, 127] (value 1 and 0) with absmax = max."""
    w = arr(1.0, 1.0)
    codes, absmax = np.array([127, 127], np.uint8), np.zeros(1, F)
    oracle.sgd_step(w, arr(0.5, 0.0), codes, absmax, 0.25, 0.5, 0.0, 1, 2)
    assert w.tolist() == [0.875, 1.0] and codes.tolist() == [255, 127] and absmax.tolist() == [0.5]
    oracle.sgd_step(w, arr(0.25, 0.0), codes, absmax, 0.25, 0.5, 0.0, 2, 2)
    assert w.tolist() == [0.75, 1.0] and codes.tolist() == [255, 127] and absmax.tolist() == [0.5]
    oracle.sgd_step(w, arr(-1.25, 0.0), codes, absmax, 0.25, 0.5, 0.0, 3, 2)   # m = 0.25 - 1.25 = -1
    assert w.tolist() == [1.0, 1.0] and codes.tolist() == [0, 127] and absmax.tolist() == [1.0]


def test_8bit_adam_with_exactly_representable_states():
    w = arr(1.0, 1.0)
    mc, ma = np.array([127, 127], np.uint8), np.zeros(1, F)
    rc, ra = np.array([0, 0], np.uint8), np.zeros(1, F)
    oracle.adam_step(w, arr(0.5, 0.0), mc, ma, rc, ra, 0.25, 0.5, 0.75, 0.0, 0.0, 1, 2, flags=0)
    assert mc.tolist() == [255, 127] and ma.tolist() == [0.25]
    assert rc.tolist() == [255, 0] and ra.tolist() == [0.0625]
    # second element: m = 0, r = 0, eps = 0 -> 0/0 would be NaN; its update uses eps > 0 below
    assert w[0] == 0.75
    w = arr(0.75, 1.0)
    oracle.adam_step(w, arr(-0.5, 0.0), mc, ma, rc, ra, 0.25, 0.5, 0.75, 1.0, 0.0, 2, 2, flags=0)
    # m = 0.125 - 0.25 = -0.125 ; r = 0.75*0.0625 + 0.0625 = 0.109375
    assert mc.tolist() == [0, 127] and ma.tolist() == [0.125]
    assert rc.tolist() == [255, 0] and ra.tolist() == [0.109375]
    assert np.allclose(w, [0.75 + 0.25 * 0.125 / (np.sqrt(0.109375) + 1.0), 1.0], rtol=2e-7)


def test_8bit_step_is_dequantize_update_quantize():
    """The step uses the fp32 states BEFORE requantization for the weight update, and both
    Adam states go through their own table (signed m, unsigned r)."""
    rng = np.random.default_rng(41)
    n, B = 3 * 256 + 17, 256
    w0 = rng.normal(0, 0.02, n).astype(F)
    m0 = rng.normal(0, 1e-3, n).astype(F)
    r0 = (rng.normal(0, 1e-3, n) ** 2).astype(F)
    g = rng.normal(0, 1e-3, n).astype(F)
    mc, ma = oracle.quantize_blockwise(m0, B, True)
    rc, ra = oracle.quantize_blockwise(r0, B, False)
    w, m, r = w0.copy(), oracle.dequantize_blockwise(mc, ma, B, True), oracle.dequantize_blockwise(rc, ra, B, False)
    oracle.adam_update_fp32(w, g, m, r, 1e-3, 0.9, 0.999, 1e-8, 0.01, 7)
    mc2, ma2 = oracle.quantize_blockwise(m, B, True)
    rc2, ra2 = oracle.quantize_blockwise(r, B, False)
    w8, mc8, ma8, rc8, ra8 = w0.copy(), mc.copy(), ma.copy(), rc.copy(), ra.copy()
    oracle.adam_step(w8, g, mc8, ma8, rc8, ra8, 1e-3, 0.9, 0.999, 1e-8, 0.01, 7, B)
    assert np.array_equal(w8, w)
    assert np.array_equal(mc8, mc2) and np.array_equal(ma8, ma2)
    assert np.array_equal(rc8, rc2) and np.array_equal(ra8, ra2)
    # SGD likewise
    w, m = w0.copy(), oracle.dequantize_blockwise(mc, ma, B, True)
    oracle.sgd_update_fp32(w, g, m, 0.1, 0.9, 1e-4)
    mc2, ma2 = oracle.quantize_blockwise(m, B, True)
    w8, mc8, ma8 = w0.copy(), mc.copy(), ma.copy()
    oracle.sgd_step(w8, g, mc8, ma8, 0.1, 0.9, 1e-4, 3, B)
    assert np.array_equal(w8, w) and np.array_equal(mc8, mc2) and np.array_equal(ma8, ma2)


def test_first_adam_step_closed_form_flat_tensor():
    """Configuration 1 (1,048,576 elements, one AdamW step from zero state, wd 0): the step does
    not depend on the quantizer.  w_1 = w_0 - lr g/(|g|+eps); the new absmax per block is
    fl((1-beta1) max|g|) and fl((1-beta2) fl(max|g|^2)) because scaling by a positive constant
    and squaring are monotone in |g|."""
    c = synth.ADAM_FLAT_SMALL
    n, B = c["n"], c["block_size"]
    w0, g = (t.numpy() for t in synth.flat_adam_inputs(n, c["seed"]))
    w = w0.copy()
    mc, ma = np.full(n, 127, np.uint8), np.zeros(n // B, F)
    rc, ra = np.zeros(n, np.uint8), np.zeros(n // B, F)
    oracle.adam_step(w, g, mc, ma, rc, ra, c["lr"], c["beta1"], c["beta2"], c["eps"],
                     c["weight_decay"], 1, B)
    g64 = g.astype(np.float64)
    want = w0.astype(np.float64) - c["lr"] * g64 / (np.abs(g64) + c["eps"])
    assert np.max(np.abs(w - want)) <= 4e-7 * np.max(np.abs(want)) + 1e-10
    moved = np.abs(w.astype(np.float64) - w0)       # ~lr each, less only where |g| ~ eps
    assert np.all(moved <= c["lr"] * 1.002) and np.mean(moved >= c["lr"] * 0.998) > 0.99
    gmax = np.max(np.abs(g).reshape(-1, B), axis=1)
    omb1 = F(1.0) - F(c["beta1"])
    omb2 = F(1.0) - F(c["beta2"])
    assert np.array_equal(ma, omb1 * gmax)
    assert np.array_equal(ra, omb2 * (gmax * gmax))
    # the element carrying the block maximum gets the end code of each table
    idx = np.argmax(np.abs(g).reshape(-1, B), axis=1) + np.arange(n // B) * B
    assert np.all((mc[idx] == 255) | (mc[idx] == 0)) and np.all(rc[idx] == 255)
    assert np.array_equal(mc[idx] == 255, g[idx] > 0)


def test_second_moment_flush_is_a_property_of_the_method():
    """An element far below its block's maximum loses its second moment to code 0."""
    n = 2048
    g = np.full(n, 1e-6, F)
    g[0] = 1.0
    w = np.zeros(n, F)
    mc, ma = np.full(n, 127, np.uint8), np.zeros(1, F)
    rc, ra = np.zeros(n, np.uint8), np.zeros(1, F)
    oracle.adam_step(w, g, mc, ma, rc, ra, 1e-3, 0.9, 0.999, 1e-8, 0.0, 1, n)
    assert rc[0] == 255 and np.all(rc[1:] == 0)              # (1e-6)^2 / 1 = 1e-12 << 1e-7
    assert np.all(mc[1:] == 129)                              # 1e-6 is the smallest signed magnitude


def test_bf16_gradients_are_widened_exactly():
    n, B = 1000, 256
    gb = synth.normal(n, 1e-3, 51, dtype=torch.bfloat16)
    g16 = gb.view(torch.int16).numpy().view(np.uint16)
    g32 = gb.float().numpy()
    w0 = synth.normal(n, 0.02, 52).numpy()
    outs = []
    for g in (g16, g32):
        w, mc, ma = w0.copy(), np.full(n, 127, np.uint8), np.zeros(4, F)
        rc, ra = np.zeros(n, np.uint8), np.zeros(4, F)
        oracle.adam_step(w, g, mc, ma, rc, ra, 1e-3, 0.9, 0.999, 1e-8, 0.05, 1, B)
        outs.append((w, mc, ma, rc, ra))
    for a, b in zip(*outs):
        assert np.array_equal(a, b)


def test_multi_tensor_is_per_tensor_and_blocks_do_not_span_tensors():
    sizes = [5, 300, 2048, 2049]
    B = 256
    rng = np.random.default_rng(61)
    ws = [rng.normal(0, 0.02, s).astype(F) for s in sizes]
    gs = [rng.normal(0, 1e-3, s).astype(F) for s in sizes]
    mcs = [np.full(s, 127, np.uint8) for s in sizes]
    mas = [np.zeros(oracle.num_blocks(s, B), F) for s in sizes]
    ws2 = [w.copy() for w in ws]
    oracle.sgd_step_multi(ws, gs, mcs, mas, 0.1, 0.9, 1e-4, 1, B)
    for t, s in enumerate(sizes):
        mc, ma = np.full(s, 127, np.uint8), np.zeros(oracle.num_blocks(s, B), F)
        oracle.sgd_step(ws2[t], gs[t], mc, ma, 0.1, 0.9, 1e-4, 1, B)
        assert np.array_equal(ws2[t], ws[t]) and np.array_equal(mc, mcs[t]) and np.array_equal(ma, mas[t])


# ------------------------------------------------------------------------------------------
# sanity bound on the quantized trajectory
# ------------------------------------------------------------------------------------------
def _curved_problem(n):
    """A noisy quadratic with per-element curvature: the gradient depends on the parameters, so
    an error in the states feeds back into the trajectory."""
    target = synth.normal(n, 0.02, 8)
    rng = np.random.default_rng(1)
    scale = torch.from_numpy(np.exp(rng.normal(0, 1, n)).astype(F))
    return lambda w, t: scale * (w - target) * 0.05 + synth.normal(n, 1e-3, 9000 + t)


def test_8bit_adam_trajectory_stays_near_the_fp32_optimizer(paper_facts):
    """The paper's claim is that 8-bit states do not change training (its evidence is recognition
    accuracy, which cannot be reproduced here).  As a sanity bound, 100 steps of the 8-bit AdamW
    checker stay within a few percent of torch's fp32 AdamW, measured against how far the
    parameters moved (measured: 3.4 % in L2, 1.6 % at the median; the gates are loose)."""
    n, B, steps = 64 * 2048, 2048, 100
    lr, b1, b2, eps = 1e-3, float(F(0.9)), float(F(0.999)), 1e-8
    wd = paper_facts["adamw_weight_decay"]
    grad = _curved_problem(n)
    w0 = synth.normal(n, 0.02, 7)
    p = torch.nn.Parameter(w0.clone())
    opt = torch.optim.AdamW([p], lr=lr, betas=(b1, b2), eps=eps, weight_decay=wd)
    w8 = w0.numpy().copy()
    nb = n // B
    mc, ma = np.full(n, 127, np.uint8), np.zeros(nb, F)
    rc, ra = np.zeros(n, np.uint8), np.zeros(nb, F)
    for t in range(1, steps + 1):
        p.grad = grad(p.detach(), t)
        opt.step()
        g8 = grad(torch.from_numpy(w8), t).numpy().astype(F)
        oracle.adam_step(w8, g8, mc, ma, rc, ra, lr, b1, b2, eps, wd, t, B)
    w32 = p.detach().numpy()
    moved = w32 - w0.numpy()
    gap = w8 - w32
    assert np.linalg.norm(gap) <= 0.10 * np.linalg.norm(moved)
    assert np.median(np.abs(gap)) <= 0.05 * np.median(np.abs(moved))


def test_8bit_sgd_trajectory_stays_near_the_fp32_optimizer(paper_facts):
    n, B, steps = 64 * 2048, 2048, 100
    lr, beta, wd = 0.01, paper_facts["sgd_momentum"], paper_facts["sgd_weight_decay"]
    grad = _curved_problem(n)
    w0 = synth.normal(n, 0.02, 7)
    p = torch.nn.Parameter(w0.clone())
    opt = torch.optim.SGD([p], lr=lr, momentum=beta, weight_decay=wd)
    w8 = w0.numpy().copy()
    mc, ma = np.full(n, 127, np.uint8), np.zeros(n // B, F)
    for t in range(1, steps + 1):
        p.grad = grad(p.detach(), t)
        opt.step()
        g8 = grad(torch.from_numpy(w8), t).numpy().astype(F)
        oracle.sgd_step(w8, g8, mc, ma, lr, beta, wd, t, B)
    w32 = p.detach().numpy()
    moved = w32 - w0.numpy()
    gap = w8 - w32
    assert np.linalg.norm(gap) <= 0.10 * np.linalg.norm(moved)
    assert np.median(np.abs(gap)) <= 0.05 * np.median(np.abs(moved))

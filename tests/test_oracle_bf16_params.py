"""Pins for the bfloat16-parameter variant of the CPU checker (no 32-bit master copy): the stored
parameter is widened exactly, Eq. sgd / Eq. adam run in binary32, and the result is rounded once,
to nearest even, when stored.  No CUDA here."""
import numpy as np
import torch

import oracle

F = np.float32


def bf(x):
    """bit patterns (uint16) of exactly representable values"""
    a = np.asarray(x, F)
    u = a.view(np.uint32)
    assert np.all((u & 0xFFFF) == 0), "not a bfloat16 value"
    return (u >> 16).astype(np.uint16)


def widen(h):
    return (np.asarray(h, np.uint16).astype(np.uint32) << 16).view(F)


def test_bf16_rounding_hand_cases():
    """bfloat16 keeps 8 significand bits: one ulp at 1.0 is 2^-7.  Half-way cases go to the even
    neighbour, everything else to the nearer one."""
    x = np.array([1.0, 1 + 2.0 ** -8, 1 + 3 * 2.0 ** -8, 1 + 2.0 ** -8 + 2.0 ** -20,
                  1 + 2.0 ** -8 - 2.0 ** -20, -(1 + 3 * 2.0 ** -8), 0.0, 3.0e38], F)
    got = widen(oracle.bf16_round(x))
    want = np.array([1.0, 1.0, 1 + 2.0 ** -6, 1 + 2.0 ** -7, 1.0, -(1 + 2.0 ** -6), 0.0, 3.0e38], F)
    assert np.array_equal(got[:7], want[:7])
    assert abs(float(got[7]) - 3.0e38) <= 3.0e38 * 2.0 ** -8


def test_bf16_rounding_is_the_identity_on_bf16_values_and_monotone():
    h = np.arange(0, 0x7F80, dtype=np.uint16)            # every finite non-negative bfloat16
    assert np.array_equal(oracle.bf16_round(widen(h)), h)
    assert np.array_equal(oracle.bf16_round(-widen(h)), h | np.uint16(0x8000))
    rng = np.random.default_rng(0)
    x = np.sort(rng.standard_normal(200000).astype(F) * 3)
    assert np.all(np.diff(widen(oracle.bf16_round(x))) >= 0)
    # nearest: the rounded value is never farther than half a bfloat16 ulp
    r = widen(oracle.bf16_round(x)).astype(np.float64)
    ulp = 2.0 ** (np.floor(np.log2(np.abs(x.astype(np.float64)))) - 7)
    assert np.all(np.abs(r - x) <= ulp / 2)


def test_bf16_rounding_equals_the_library_conversion():
    rng = np.random.default_rng(1)
    x = (rng.standard_normal(1 << 18) * 10.0 ** rng.integers(-20, 20, 1 << 18)).astype(F)
    want = torch.from_numpy(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(oracle.bf16_round(x), want)


def test_sgd_with_bf16_parameters_hand_computed():
    """lr = 1, momentum = 0, no decay: w' = w - g in binary32, then one rounding to bfloat16.
    w = 1: g = -2^-8 lands half-way between 1 and 1 + 2^-7 and goes to the even 1;
    g = -3*2^-8 lands half-way between 1 + 2^-7 and 1 + 2^-6 and goes to the even 1 + 2^-6;
    g = -(2^-8 + 2^-16) is past the half and goes up to 1 + 2^-7."""
    g = np.array([-2.0 ** -8, -3 * 2.0 ** -8, -(2.0 ** -8 + 2.0 ** -16), 0.5], F)
    w = bf([1.0, 1.0, 1.0, 1.0])
    mc, ma = np.full(4, 127, np.uint8), np.zeros(1, F)
    oracle.sgd_step(w, g, mc, ma, 1.0, 0.0, 0.0, 1, 256)
    assert widen(w).tolist() == [1.0, 1 + 2.0 ** -6, 1 + 2.0 ** -7, 0.5]
    assert ma[0] == 0.5                                       # the state is that of the fp32 run


def test_bf16_parameter_step_is_the_fp32_step_on_the_widened_parameter_rounded_once():
    rng = np.random.default_rng(2)
    n, B = 5 * 256 + 17, 256
    w16 = oracle.bf16_round((rng.standard_normal(n) * 0.02).astype(F))
    g = (rng.standard_normal(n) * 1e-3).astype(F)
    hp = (1e-3, 0.9, 0.999, 1e-8, 0.01)
    a_w, b_w = w16.copy(), widen(w16).copy()
    st = lambda: (np.full(n, 127, np.uint8), np.zeros(oracle.num_blocks(n, B), F),
                  np.zeros(n, np.uint8), np.zeros(oracle.num_blocks(n, B), F))
    sa, sb = st(), st()
    oracle.adam_step(a_w, g, *sa, *hp, 1, B)
    oracle.adam_step(b_w, g, *sb, *hp, 1, B)
    assert np.array_equal(a_w, oracle.bf16_round(b_w))
    for u, v in zip(sa, sb):
        assert np.array_equal(u, v)
    # coupled decay reads the widened parameter too
    a_w, b_w = w16.copy(), widen(w16).copy()
    ma, mb = (np.full(n, 127, np.uint8), np.zeros(oracle.num_blocks(n, B), F)), \
             (np.full(n, 127, np.uint8), np.zeros(oracle.num_blocks(n, B), F))
    oracle.sgd_step(a_w, g, *ma, 0.1, 0.9, 0.5, 1, B)
    oracle.sgd_step(b_w, g, *mb, 0.1, 0.9, 0.5, 1, B)
    assert np.array_equal(a_w, oracle.bf16_round(b_w))
    assert np.array_equal(ma[0], mb[0]) and np.array_equal(ma[1], mb[1])

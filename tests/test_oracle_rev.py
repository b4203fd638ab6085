"""Pins of the CPU checker for the reversible-network memory kernels (Section III-B): additive
coupling (Eq. revnet4), its inverse (Eq. revnet5) and the invertible down-sampling (Eq. revnet6).
Nothing here touches the CUDA path."""
import os

import numpy as np
import pytest
import torch

from oracle import rev

F32 = np.float32
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _golden(name):
    """Reads 'key: numbers' lines of a golden text file."""
    out = {}
    with open(os.path.join(ROOT, "tests", "golden", name)) as fh:
        for line in fh:
            line = line.split("#", 1)[0].strip()
            if not line:
                continue
            key, val = line.split(":", 1)
            out[key.strip()] = [float(v) for v in val.split()]
    return out


# ------------------------------------------------------------------------------------------------
# Eq. revnet6: C x F x T -> r^2 C x F/r x T/r
# ------------------------------------------------------------------------------------------------
def test_space_to_depth_hand_computed_case():
    """A 2 x 2 x 4 tensor worked by hand from the description in Section III-B: every channel is
    cut into 2 x 2 blocks and each C x 2 x 2 block is flattened into 4C x 1 x 1."""
    g = _golden("space_to_depth_2x2x4.txt")
    x = np.array(g["input"], F32).reshape(1, 2, 2, 4)
    y = rev.space_to_depth(x, 2)
    assert y.shape == (1, 8, 1, 2)
    assert y.ravel().tolist() == g["output"]
    assert rev.depth_to_space(y, 2).ravel().tolist() == g["input"]


def test_space_to_depth_shape_and_block_content():
    """Output shape r^2 C x F/r x T/r (Eq. revnet6), and the r*r output channels that belong to
    input channel c hold, at (fo, to), exactly the r x r block of that channel at (r*fo, r*to)."""
    rng = np.random.default_rng(0)
    for (n, c, f, t, r) in ((2, 3, 4, 6, 2), (1, 5, 8, 10, 2), (2, 2, 6, 9, 3), (1, 1, 2, 2, 2)):
        x = rng.standard_normal((n, c, f, t)).astype(F32)
        y = rev.space_to_depth(x, r)
        assert y.shape == (n, r * r * c, f // r, t // r)
        for cc in range(c):
            for fo in range(f // r):
                for to in range(t // r):
                    block = x[:, cc, r * fo:r * fo + r, r * to:r * to + r].reshape(n, r * r)
                    assert np.array_equal(y[:, cc * r * r:(cc + 1) * r * r, fo, to], block)


def test_space_to_depth_is_a_bijection_with_the_stated_inverse():
    """The rearrangement keeps every element exactly once (Section III-B: same number of elements,
    reversible), and depth_to_space undoes it bit for bit, both ways round."""
    n, c, f, t = 2, 3, 6, 10
    x = np.arange(n * c * f * t, dtype=F32).reshape(n, c, f, t)
    y = rev.space_to_depth(x, 2)
    assert np.array_equal(np.sort(y.ravel()), x.ravel())
    assert np.array_equal(rev.depth_to_space(y, 2), x)
    z = np.arange(n * 4 * c * 3 * 5, dtype=F32).reshape(n, 4 * c, 3, 5)
    assert np.array_equal(rev.space_to_depth(rev.depth_to_space(z, 2), 2), z)


def test_space_to_depth_equals_the_library_routine_of_the_row_major_reading():
    """torch's pixel_unshuffle implements the same row-major flattening of the C x r x r block."""
    rng = np.random.default_rng(1)
    for (n, c, f, t, r) in ((2, 6, 8, 12, 2), (1, 3, 10, 50, 2), (1, 2, 9, 6, 3)):
        x = rng.standard_normal((n, c, f, t)).astype(F32)
        want = torch.nn.functional.pixel_unshuffle(torch.from_numpy(x), r).numpy()
        assert np.array_equal(rev.space_to_depth(x, r), want)
        assert np.array_equal(rev.depth_to_space(want, r),
                              torch.nn.functional.pixel_shuffle(torch.from_numpy(want), r).numpy())


def test_space_to_depth_rejects_sizes_that_do_not_divide():
    with pytest.raises(ValueError):
        rev.space_to_depth(np.zeros((1, 1, 3, 4), F32), 2)
    with pytest.raises(ValueError):
        rev.depth_to_space(np.zeros((1, 6, 2, 2), F32), 2)


# ------------------------------------------------------------------------------------------------
# Eq. revnet4 / revnet5: additive coupling
# ------------------------------------------------------------------------------------------------
def _affine(a, b):
    return lambda v: (a * v.astype(np.float64) + b).astype(F32)


def test_coupling_hand_computed_case():
    """One sample, two channels of one element: x1 = 3, x2 = 5, F(v) = 2v + 1, G(v) = v - 4.
    Eq. revnet4: y1 = 3 + F(5) = 14, y2 = 5 + G(14) = 15.  Eq. revnet5 recovers (3, 5)."""
    x = np.array([3.0, 5.0], F32).reshape(1, 2, 1, 1)
    Fb, Gb = _affine(2, 1), _affine(1, -4)
    y = rev.rev_block_forward(x, Fb, Gb)
    assert y.ravel().tolist() == [14.0, 15.0]
    assert rev.rev_block_inverse(y, Fb, Gb).ravel().tolist() == [3.0, 5.0]


def test_coupling_uses_y1_for_g_and_the_right_halves():
    """G must see y1 (not x1) and F must see x2 (the upper channel half): with branches that are
    not interchangeable, the closed form of Eq. revnet4 is reproduced element by element."""
    rng = np.random.default_rng(2)
    x = rng.integers(-50, 50, (3, 4, 2, 5)).astype(F32)      # small integers: every sum is exact
    Fb, Gb = _affine(3, 7), _affine(-2, 1)
    y = rev.rev_block_forward(x, Fb, Gb)
    x1, x2 = x[:, :2].astype(np.float64), x[:, 2:].astype(np.float64)
    y1 = x1 + (3 * x2 + 7)
    y2 = x2 + (-2 * y1 + 1)
    assert np.array_equal(y[:, :2], y1.astype(F32)) and np.array_equal(y[:, 2:], y2.astype(F32))
    assert np.array_equal(rev.rev_block_inverse(y, Fb, Gb), x)   # exact arithmetic: exact inverse


def test_coupling_is_one_binary32_operation_per_element():
    rng = np.random.default_rng(3)
    a = rng.standard_normal((2, 6, 3, 7)).astype(F32)
    t = (rng.standard_normal((2, 3, 3, 7)) * 10).astype(F32)
    for which in (0, 1):
        lo, hi = (0, 3) if which == 0 else (3, 6)
        for sign in (+1, -1):
            out = np.full_like(a, np.nan)
            rev.couple_half(a, t, out, which, sign)
            want = (a[:, lo:hi] + t) if sign > 0 else (a[:, lo:hi] - t)     # numpy float32 arithmetic
            assert np.array_equal(out[:, lo:hi], want)
            other = out[:, 3:] if which == 0 else out[:, :3]
            assert np.all(np.isnan(other)), "the other half must not be written"


def test_coupling_inverse_recovers_the_input_to_rounding():
    """x1' = fl(fl(x1 + f) - f) differs from x1 by at most half an ulp of y1 plus half an ulp of
    x1' (two roundings), and is exact whenever x1 + f is representable."""
    rng = np.random.default_rng(4)
    x = rng.standard_normal((2, 8, 4, 6)).astype(F32)
    Fb = lambda v: np.tanh(v * 3).astype(F32) * 5
    Gb = lambda v: (np.sin(v) * 2).astype(F32)
    y = rev.rev_block_forward(x, Fb, Gb)
    xr = rev.rev_block_inverse(y, Fb, Gb)
    eps = 2.0 ** -24
    # x2 first: y2 -> x2' uses the same G(y1) on both sides
    err2 = np.abs(xr[:, 4:].astype(np.float64) - x[:, 4:])
    assert np.all(err2 <= eps * (np.abs(y[:, 4:]) + np.abs(xr[:, 4:])) * 1.0000001)
    # x1 is recovered through F(x2'), so only compare where x2' == x2 exactly
    same = xr[:, 4:] == x[:, 4:]
    err1 = np.abs(xr[:, :4].astype(np.float64) - x[:, :4])
    bound1 = eps * (np.abs(y[:, :4]) + np.abs(xr[:, :4])) * 1.0000001
    assert np.all((err1 <= bound1) | ~same)
    assert same.any()
    # sums that are representable come back exactly (dyadic values of a few bits)
    xd = (rng.integers(-64, 64, (1, 4, 3, 5)) / 8.0).astype(F32)
    Fd = lambda v: (v * 0.5 + 0.25).astype(F32)
    Gd = lambda v: (v * 0.25 - 1.0).astype(F32)
    assert np.array_equal(rev.rev_block_inverse(rev.rev_block_forward(xd, Fd, Gd), Fd, Gd), xd)


# ------------------------------------------------------------------------------------------------
# Alg. 1: the gradients a reversible block must return
# ------------------------------------------------------------------------------------------------
class _Scale(torch.nn.Module):
    """A branch with one parameter: v -> a * v."""

    def __init__(self, a):
        super().__init__()
        self.a = torch.nn.Parameter(torch.tensor(float(a)))

    def forward(self, v):
        return self.a * v


def test_block_gradients_closed_form_for_scalar_branches():
    """With F(v) = a v and G(v) = b v, Eq. revnet4 gives y1 = x1 + a x2, y2 = x2 + b y1, hence
    dL/dx1 = dy1 + b dy2, dL/dx2 = a (dy1 + b dy2) + dy2, dL/da = sum((dy1 + b dy2) x2),
    dL/db = sum(dy2 y1): the quantities Alg. 1 returns."""
    a, b = 0.75, -1.5
    g = torch.Generator().manual_seed(5)
    x = torch.randn(2, 4, 3, 5, generator=g, dtype=torch.float64)
    dy = torch.randn(2, 4, 3, 5, generator=g, dtype=torch.float64)
    y, dx, dwf, dwg = rev.rev_block_gradients(x, _Scale(a), _Scale(b), dy)
    x1, x2, dy1, dy2 = x[:, :2], x[:, 2:], dy[:, :2], dy[:, 2:]
    y1 = x1 + a * x2
    dz1 = dy1 + b * dy2
    assert torch.allclose(y, torch.cat([y1, x2 + b * y1], 1), rtol=0, atol=1e-14)
    assert torch.allclose(dx[:, :2], dz1, rtol=0, atol=1e-14)
    assert torch.allclose(dx[:, 2:], a * dz1 + dy2, rtol=0, atol=1e-14)
    assert abs(float(dwf[0]) - float((dz1 * x2).sum())) < 1e-12
    assert abs(float(dwg[0]) - float((dy2 * y1).sum())) < 1e-12


def test_block_gradients_match_finite_differences_for_conv_branches():
    torch.manual_seed(6)
    mk = lambda: torch.nn.Sequential(torch.nn.Conv2d(2, 2, 3, padding=1), torch.nn.Tanh(),
                                     torch.nn.Conv2d(2, 2, 3, padding=1))
    Fm, Gm = mk().double(), mk().double()
    x = torch.randn(1, 4, 3, 4, dtype=torch.float64)
    dy = torch.randn(1, 4, 3, 4, dtype=torch.float64)
    _, dx, dwf, _ = rev.rev_block_gradients(x, Fm, Gm, dy)

    def loss(xx):
        y1 = xx[:, :2] + Fm(xx[:, 2:])
        return float((torch.cat([y1, xx[:, 2:] + Gm(y1)], 1) * dy).sum())
    h = 1e-6
    for idx in ((0, 0, 1, 2), (0, 3, 2, 0), (0, 2, 0, 3)):
        e = torch.zeros_like(x)
        e[idx] = h
        fd = (loss(x + e) - loss(x - e)) / (2 * h)
        assert abs(fd - float(dx[idx])) < 1e-6 * max(1.0, abs(fd))
    w = next(Fm.parameters())
    with torch.no_grad():
        w0 = float(w[0, 1, 1, 1])
        w[0, 1, 1, 1] = w0 + h
        up = loss(x)
        w[0, 1, 1, 1] = w0 - h
        dn = loss(x)
        w[0, 1, 1, 1] = w0
    assert abs((up - dn) / (2 * h) - float(dwf[0][0, 1, 1, 1])) < 1e-6

"""Pins for the CPU checker's code book (Section IV-B, Fig. dynamic_tree).

Nothing here calls the CUDA path.  The checks are structural facts of the four-part bit
format the paper describes, an independent decode of the bit string in exact rational
arithmetic, and the numbers the paper prints.
"""
from fractions import Fraction

import numpy as np
import pytest

import oracle


def f32_exact(fr: Fraction) -> np.float32:
    """Fraction -> nearest float32 (via the nearest float64; innocuous for these values)."""
    return np.float32(float(fr))


def decode_bit_string(bits: str) -> Fraction:
    """Value of a magnitude field given as a bit string, straight from the description:
    a run of zeros (decimal exponent), an indicator 1, then a linear fraction."""
    if "1" not in bits:
        return Fraction(0)
    zeros = bits.index("1")
    frac_bits = bits[zeros + 1:]
    levels = 2 ** len(frac_bits)
    k = int(frac_bits, 2) if frac_bits else 0
    # decade (10^-(zeros+1), 10^-zeros], cut into `levels` equal steps, upper end included
    lo = Fraction(1, 10 ** (zeros + 1))
    hi = Fraction(1, 10 ** zeros)
    return lo + (hi - lo) * Fraction(k + 1, levels)


@pytest.fixture(scope="module")
def Qs():
    return oracle.codebook(True)


@pytest.fixture(scope="module")
def Qu():
    return oracle.codebook(False)


def test_shape_order_endpoints(Qs, Qu, paper_facts):
    assert Qs.shape == (256,) and Qu.shape == (256,)
    assert Qs.dtype == np.float32 and Qu.dtype == np.float32
    assert 2 ** int(paper_facts["code_bits"]) == 256
    assert np.all(np.diff(Qs.astype(np.float64)) >= 0)
    assert np.all(np.diff(Qu.astype(np.float64)) > 0)
    assert Qs[0] == paper_facts["range_min"] and Qs[255] == paper_facts["range_max"]
    assert Qu[0] == 0.0 and Qu[255] == paper_facts["range_max"]
    assert (Qs == 0).sum() == 2 and Qs[127] == 0 and Qs[128] == 0   # the sign bit gives two zeros
    assert (Qu == 0).sum() == 1


def test_signed_is_symmetric(Qs):
    assert np.array_equal(Qs[::-1], -Qs)
    # apart from the doubled zero all values are distinct
    assert len(np.unique(Qs)) == 255


def test_smallest_magnitudes(Qs, Qu, paper_facts):
    # the zero run can be as long as the field minus the indicator: 6 zeros signed, 7 unsigned
    assert Qs[129] == np.float32(1e-6)
    assert Qu[1] == np.float32(paper_facts["smallest_exponent"])


@pytest.mark.parametrize("signed", [True, False])
def test_decades(signed, Qs, Qu, paper_facts):
    """Per-decade population, equal spacing, and the grid continuing into the decade below."""
    W = 7 if signed else 8
    pos = (Qs[128:] if signed else Qu).astype(np.float64)   # index = magnitude pattern
    for E in range(W):
        F = W - 1 - E
        members = [v for v in pos[1:] if 10.0 ** -(E + 1) * (1 + 1e-6) < v <= 10.0 ** -E * (1 + 1e-6)]
        assert len(members) == 2 ** F
        grid = np.array([10.0 ** -(E + 1)] + members)     # lower end point = top of decade E+1
        steps = np.diff(grid)
        assert np.allclose(steps, 0.9 * 10.0 ** -E / 2 ** F, rtol=1e-5)
        # magnitude-pattern order is value order: patterns 2^F .. 2^(F+1)-1 are this decade
        assert np.array_equal(pos[2 ** F: 2 ** (F + 1)], np.array(members))
        if E + 1 < W:
            assert np.isclose(pos[2 ** F - 1], 10.0 ** -(E + 1), rtol=1e-6)
    # "fractional precision up to 1/63": the finest field (6 bits after sign and indicator)
    # has 64 levels, i.e. 63 equal intervals between the lowest and the highest of them
    top_signed = Qs[128 + 64:]
    assert len(top_signed) - 1 == int(paper_facts["fraction_intervals"])


@pytest.mark.parametrize("signed", [True, False])
def test_values_from_bit_strings(signed, Qs, Qu):
    """Every entry equals the exactly-rounded value decoded from its own bit string."""
    W = 7 if signed else 8
    for p in range(2 ** W):
        exact = decode_bit_string(format(p, "0%db" % W))
        want = f32_exact(exact)
        if signed:
            assert Qs[128 + p] == want and Qs[127 - p] == -want
        else:
            assert Qu[p] == want
        # the stored float is within half an ulp of the rational value
        got = Fraction(float(Qs[128 + p] if signed else Qu[p]))
        if exact:
            ulp = Fraction(float(np.spacing(np.float32(float(exact)))))
            assert abs(got - exact) <= ulp / 2


def test_closed_form_rational(Qs, Qu):
    """value(E,k) = (2^F + 9(k+1)) / (10^(E+1) 2^F), checked in integer arithmetic."""
    for W, pos in ((7, Qs[128:]), (8, Qu)):
        for E in range(W):
            F = W - 1 - E
            for k in range(2 ** F):
                fr = Fraction(2 ** F + 9 * (k + 1), 10 ** (E + 1) * 2 ** F)
                assert pos[2 ** F + k] == f32_exact(fr)
    assert Qs[255] == 1.0 and Qu[255] == 1.0


def test_state_memory_saving(paper_facts):
    """8-bit codes + one fp32 absmax per block against fp32 states: the paper's 75 %."""
    B = int(paper_facts["block_size"])
    for state_bytes in (paper_facts["sgd_state_bytes_fp32"], paper_facts["adam_state_bytes_fp32"]):
        n_states = state_bytes / 4
        n = 10 * B
        codes, absmax = oracle.quantize_blockwise(np.ones(n, np.float32), B, True)
        bytes_8bit = n_states * (codes.nbytes + absmax.nbytes)
        saving = 100.0 * (1.0 - bytes_8bit / (state_bytes * n))
        assert saving == pytest.approx(100.0 * (1 - (1 + 4 / B) / 4), abs=1e-9)
        assert round(saving) == paper_facts["memory_saving_percent"]

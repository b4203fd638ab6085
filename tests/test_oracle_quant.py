"""Pins for the CPU checker's quantizer (Eq. quant1, quant2, quant3).  No CUDA here.

The exhaustive scan is the definition of Eq. quant2 and is itself pinned to numpy's argmin;
the binary search is then proven equal to it on tables, mid-points, their neighbourhoods
and random inputs.  Round trips, the error bound of the grid, block independence and the
degenerate cases pin Eq. quant1 and quant3.
"""
import numpy as np
import pytest

import oracle

TABLES = {True: oracle.codebook(True), False: oracle.codebook(False)}


def numpy_argmin(Q, v):
    """Eq. quant2 with a library routine: argmin_j |Q_j - v| in float64, lowest index on ties."""
    d = np.abs(Q.astype(np.float64)[None, :] - v.astype(np.float64)[:, None])
    return np.argmin(d, axis=1).astype(np.uint8)


def ulp_neighbourhood(x32, radius=64):
    """The binary32 numbers within `radius` ulps of each x."""
    bits = x32.astype(np.float32).view(np.int32).astype(np.int64)
    out = []
    for d in range(-radius, radius + 1):
        b = bits + d
        out.append(b.astype(np.int32).view(np.float32))
    return np.concatenate(out)


@pytest.mark.parametrize("signed", [True, False])
def test_scan_is_the_definition(signed):
    Q = TABLES[signed]
    rng = np.random.default_rng(10)
    v = np.concatenate([rng.uniform(-1, 1, 20000), rng.normal(0, 1e-4, 5000), Q,
                        10.0 ** rng.uniform(-9, 0, 5000)]).astype(np.float32)
    assert np.array_equal(oracle.nearest(Q, v, "scan"), numpy_argmin(Q, v))


@pytest.mark.parametrize("signed", [True, False])
def test_bsearch_equals_scan(signed):
    Q = TABLES[signed]
    rng = np.random.default_rng(11)
    mids = ((Q[:-1].astype(np.float64) + Q[1:].astype(np.float64)) / 2).astype(np.float32)
    pools = [
        Q, ulp_neighbourhood(Q), ulp_neighbourhood(mids),
        rng.uniform(-1, 1, 2_000_000).astype(np.float32),
        (10.0 ** rng.uniform(-10, 0, 500_000) * rng.choice([-1, 1], 500_000)).astype(np.float32),
        np.array([0.0, -0.0, 1.0, -1.0, 1.5, -1.5, 1e-30, -1e-30, 4.9e-7, 5.1e-7, 4.9e-8, 5.1e-8],
                 np.float32),
    ]
    for v in pools:
        v = v[np.isfinite(v)]
        assert np.array_equal(oracle.nearest(Q, v, "bsearch"), oracle.nearest(Q, v, "scan"))


@pytest.mark.parametrize("signed", [True, False])
def test_exact_ties_take_the_lower_index(signed):
    """Mid-points that are themselves binary32 numbers are true ties of Eq. quant2."""
    Q = TABLES[signed].astype(np.float64)
    mids64 = (Q[:-1] + Q[1:]) / 2
    mids32 = mids64.astype(np.float32)
    exact = np.nonzero((mids32.astype(np.float64) == mids64) & (Q[:-1] != Q[1:]))[0]
    assert len(exact) > 10                      # such ties exist, so the rule matters
    got = oracle.nearest(TABLES[signed], mids32[exact], "bsearch")
    want = exact.astype(np.uint8)
    if signed:
        want[want == 128] = 127               # the tie between +0 and 1e-6 goes to the first zero
    assert np.array_equal(got, want)
    assert np.array_equal(got, oracle.nearest(TABLES[signed], mids32[exact], "scan"))


@pytest.mark.parametrize("signed", [True, False])
def test_monotone_and_fixed_points(signed):
    Q = TABLES[signed]
    v = np.sort(np.random.default_rng(12).uniform(-1.1, 1.1, 300000).astype(np.float32))
    c = oracle.nearest(Q, v).astype(np.int32)
    assert np.all(np.diff(c) >= 0)
    # every table value is its own nearest code (the lower of the two zeros for 0)
    want = np.arange(256, dtype=np.uint8)
    if signed:
        want[128] = 127
    assert np.array_equal(oracle.nearest(Q, Q), want)
    if signed:
        assert 128 not in set(oracle.nearest(Q, v).tolist())
    else:
        assert np.all(oracle.nearest(Q, -np.abs(v)) == 0)      # negative input -> value 0


@pytest.mark.parametrize("signed", [True, False])
@pytest.mark.parametrize("N", [1.0, 3.7e-5, 2.0 ** -20, 1e4])
def test_round_trip_of_every_code(signed, N):
    """quantize(dequantize(codes, N)) gives the codes back (128 comes back as 127)."""
    codes = np.arange(256, dtype=np.uint8)
    absmax = np.array([N], np.float32)
    x = oracle.dequantize_blockwise(codes, absmax, 256, signed)
    assert np.array_equal(x, TABLES[signed] * np.float32(N))          # Eq. quant3, one multiply
    codes2, absmax2 = oracle.quantize_blockwise(x, 256, signed)
    want = codes.copy()
    if signed:
        want[128] = 127
    assert np.array_equal(codes2, want)
    assert absmax2[0] == np.float32(N)


@pytest.mark.parametrize("signed", [True, False])
@pytest.mark.parametrize("B", [256, 2048, 4096])
def test_requantizing_is_idempotent_and_absmax(signed, B):
    rng = np.random.default_rng(13)
    n = 5 * B + 37                                   # ragged last block
    x = rng.laplace(0, 1, n).astype(np.float32)
    x[rng.random(n) < 1e-3] *= 100
    if not signed:
        x = np.abs(x)
    codes, absmax = oracle.quantize_blockwise(x, B, signed)
    nb = (n + B - 1) // B
    assert absmax.shape == (nb,)
    for b in range(nb):                               # Eq. quant1: N_b = max |T_b|
        assert absmax[b] == np.max(np.abs(x[b * B:(b + 1) * B]))
    top = 255
    for b in range(nb):                               # the absmax element normalises to exactly 1
        blk = slice(b * B, min(n, (b + 1) * B))
        i = np.argmax(np.abs(x[blk]))
        assert codes[blk][i] in ((top, 0) if signed else (top,))
    y = oracle.dequantize_blockwise(codes, absmax, B, signed)
    codes2, absmax2 = oracle.quantize_blockwise(y, B, signed)
    assert np.array_equal(codes2, codes) and np.array_equal(absmax2, absmax)
    # the scan-based block quantizer gives the same codes
    codes3, _ = oracle.quantize_blockwise(x, B, signed, method="scan")
    assert np.array_equal(codes3, codes)


@pytest.mark.parametrize("signed", [True, False])
def test_error_bound_of_the_grid(signed):
    """|dequant(quant(x)) - x| <= N_b * half a grid step of the decade x/N_b falls in."""
    W = 7 if signed else 8
    B = 2048
    rng = np.random.default_rng(14)
    x = (10.0 ** rng.uniform(-9, 0, 40 * B) * (rng.choice([-1, 1], 40 * B) if signed else 1.0))
    x = x.astype(np.float32)
    codes, absmax = oracle.quantize_blockwise(x, B, signed)
    y = oracle.dequantize_blockwise(codes, absmax, B, signed).astype(np.float64)
    N = np.repeat(absmax.astype(np.float64), B)
    v = np.abs(x.astype(np.float64)) / N
    E = np.clip(np.ceil(-np.log10(np.maximum(v, 1e-300)) - 1e-12) - 1, 0, None)   # v in (10^-(E+1), 10^-E]
    # decades above the lowest: half of the uniform step; the lowest decade holds one value,
    # 10^-(W-1), whose lower neighbour is 0, so there (and below) the bound is half of it
    half_step = np.where(E < W - 1, 0.45 * 10.0 ** -E / 2.0 ** (W - 1 - np.minimum(E, W - 1)),
                         0.5 * 10.0 ** -(W - 1))
    err = np.abs(y - x.astype(np.float64))
    assert np.all(err <= N * half_step * (1 + 1e-5) + 1e-12 * N)
    # and the bound is attained to within a factor 2 somewhere, i.e. it is not slack
    assert np.max(err / (N * half_step)) > 0.5


def test_blocks_are_independent():
    rng = np.random.default_rng(15)
    B = 256
    x = rng.normal(0, 1, 7 * B + 5).astype(np.float32)
    codes, absmax = oracle.quantize_blockwise(x, B, True)
    perm = [3, 0, 6, 7, 1]                                       # reorder and drop blocks
    pieces = [x[b * B:(b + 1) * B] for b in perm if b != 7]
    x2 = np.concatenate(pieces + [x[7 * B:]])
    codes2, absmax2 = oracle.quantize_blockwise(x2, B, True)
    order = [3, 0, 6, 1, 7]
    for pos, b in enumerate(order):
        src = codes[b * B:(b + 1) * B]
        assert np.array_equal(codes2[pos * B: pos * B + len(src)], src)
        assert absmax2[pos] == absmax[b]


def test_degenerate_inputs():
    for signed, zero_code in ((True, 127), (False, 0)):
        codes, absmax = oracle.quantize_blockwise(np.zeros(300, np.float32), 256, signed)
        assert np.all(codes == zero_code) and np.all(absmax == 0)
        assert np.all(oracle.dequantize_blockwise(codes, absmax, 256, signed) == 0)
        codes, absmax = oracle.quantize_blockwise(np.zeros(0, np.float32), 256, signed)
        assert codes.size == 0 and absmax.size == 0
        codes, absmax = oracle.quantize_blockwise(np.array([-3.0], np.float32), 2048, signed)
        assert absmax[0] == 3.0 and codes[0] == (0 if signed else 0)
    # a single element block: x / |x| = +-1
    codes, absmax = oracle.quantize_blockwise(np.array([2.5, -2.5], np.float32), 1, True)
    assert codes.tolist() == [255, 0] and absmax.tolist() == [2.5, 2.5]
    with pytest.raises(ValueError):
        oracle.quantize_blockwise(np.zeros(4, np.float32), 0, True)


def division_discriminators(signed, want=32, seed=16):
    """Pairs (x, N) whose code differs between x / N (Eq. quant1 as written) and x * (1 / N)."""
    Q = TABLES[signed]
    Q64 = Q.astype(np.float64)
    mids = ((Q64[:-1] + Q64[1:]) / 2)[Q64[:-1] != Q64[1:]]
    mids = mids[mids > 0].astype(np.float32)
    rng = np.random.default_rng(seed)
    xs, Ns = [], []
    while len(xs) < want:
        N = rng.uniform(0.5, 2.0, 200000).astype(np.float32)
        T = rng.choice(mids, N.size)
        x = (T * N).astype(np.float32)                       # x / N lands within an ulp of a mid-point
        v_div = x / N
        v_rcp = x * (np.float32(1.0) / N)
        differ = oracle.nearest(Q, v_div) != oracle.nearest(Q, v_rcp)
        xs += x[differ].tolist()
        Ns += N[differ].tolist()
    return np.array(xs[:want], np.float32), np.array(Ns[:want], np.float32)


@pytest.mark.parametrize("signed", [True, False])
def test_normalisation_is_a_true_division(signed):
    """Eq. quant1 divides by N_b.  Near a mid-point of the table a reciprocal-multiply lands on
    the other code; on such inputs the block quantizer must follow the division."""
    Q = TABLES[signed]
    x, N = division_discriminators(signed)
    for xi, Ni in zip(x, N):
        codes, absmax = oracle.quantize_blockwise(np.array([xi, Ni], np.float32), 2, signed)
        assert absmax[0] == Ni and codes[1] == 255
        assert codes[0] == oracle.nearest(Q, np.array([xi / Ni], np.float32))[0]
        assert codes[0] != oracle.nearest(Q, np.array([xi * (np.float32(1.0) / Ni)], np.float32))[0]

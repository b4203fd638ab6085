"""Parity of the reversible-network kernels (Section III-B) against the CPU checker, through the
C ABI: coupling halves and the invertible down-sampling bit for bit; whole blocks with branches
evaluated identically on both sides; Alg. 1 against plain binary64 back-propagation."""
import numpy as np
import pytest
import torch

from oracle import rev as orev
import paper_2412_01195_b200 as dt8
from paper_2412_01195_b200 import rev, synth

pytestmark = pytest.mark.gpu
F32 = np.float32
DEV = "cuda"


@pytest.fixture(scope="module", autouse=True)
def _setup():
    assert torch.cuda.is_available(), "these tests need a CUDA device"
    dt8.dt8_init()
    yield
    torch.cuda.synchronize()


def act(shape, seed, scale=1.0):
    n = int(np.prod(shape))
    return (synth.normal(n, scale, seed)).reshape(shape)


# ------------------------------------------------------------------------------------------------
# coupling halves (Eq. revnet4 / revnet5)
# ------------------------------------------------------------------------------------------------
@pytest.mark.parametrize("shape", [(1, 2, 1, 1), (3, 4, 5, 7), (2, 6, 8, 50), (5, 48, 20, 50),
                                   (2, 48, 80, 200), (1, 2, 1, 4 * 1024 * 5 + 4)])
def test_coupling_halves_match_the_checker(shape):
    x = act(shape, 2000)
    t = act((shape[0], shape[1] // 2) + shape[2:], 2001, 3.0)
    for which in (0, 1):
        for name, sign in (("dt8_rev_coupling_forward", +1), ("dt8_rev_coupling_inverse", -1)):
            out = torch.full(shape, float("nan"), device=DEV)
            getattr(rev, name)(x.to(DEV), t.to(DEV), out, which)
            want = np.full(shape, np.nan, F32)
            orev.couple_half(x.numpy(), t.numpy(), want, which, sign)
            torch.cuda.synchronize()
            assert np.array_equal(out.cpu().numpy().view(np.uint32), want.view(np.uint32))


def test_coupling_in_place_and_at_four_byte_offsets():
    shape = (3, 6, 7, 9)                                   # half = 189: the scalar path
    x, t = act(shape, 2010), act((3, 3, 7, 9), 2011)
    want = x.numpy().copy()
    orev.couple_half(x.numpy(), t.numpy(), want, 1, +1)
    xg = x.to(DEV)
    rev.dt8_rev_coupling_forward(xg, t.to(DEV), xg, 1)
    assert np.array_equal(xg.cpu().numpy(), want)
    # 16-byte-divisible half but pointers only 4-byte aligned
    shape = (2, 4, 4, 8)
    n = int(np.prod(shape))
    pool = torch.full((3 * n + 64,), float("nan"), device=DEV)
    xa, ta, oa = pool[1:1 + n].view(shape), pool[n + 3:n + 3 + n // 2].view(2, 2, 4, 8), pool[2 * n + 9:3 * n + 9].view(shape)
    x, t = act(shape, 2012), act((2, 2, 4, 8), 2013)
    xa.copy_(x)
    ta.copy_(t)
    rev.dt8_rev_coupling_inverse(xa, ta, oa, 0)
    want = np.full(shape, np.nan, F32)
    orev.couple_half(x.numpy(), t.numpy(), want, 0, -1)
    assert np.array_equal(oa.cpu().numpy().view(np.uint32), want.view(np.uint32))
    assert bool(torch.isnan(pool[0])) and bool(torch.isnan(pool[2 * n + 8])) and bool(torch.isnan(pool[3 * n + 9]))


def test_coupling_argument_checks():
    x = torch.zeros(2, 4, 3, 3, device=DEV)
    with pytest.raises(ValueError):
        rev.dt8_rev_coupling_forward(x, torch.zeros(2, 2, 3, 2, device=DEV), x, 0)
    with pytest.raises(ValueError):
        rev.dt8_rev_coupling_forward(torch.zeros(2, 3, 3, 3, device=DEV), torch.zeros(9, device=DEV), x, 0)
    with pytest.raises(dt8.DT8Error):
        rev.dt8_rev_coupling_forward(x, torch.zeros(2, 2, 3, 3, device=DEV), x, 2)
    rev.dt8_rev_coupling_forward(x[:0], torch.zeros(0, 2, 3, 3, device=DEV), x[:0], 0)   # empty batch: no-op


# ------------------------------------------------------------------------------------------------
# invertible down-sampling (Eq. revnet6, r = 2)
# ------------------------------------------------------------------------------------------------
@pytest.mark.parametrize("shape", [(1, 1, 2, 2), (1, 2, 2, 4), (2, 3, 4, 6), (3, 5, 6, 10), (2, 24, 80, 200),
                                   (2, 48, 40, 100), (3, 75, 20, 50), (1, 7, 2, 2050), (4, 1, 34, 4), (2, 2, 126, 102), (5, 3, 2, 6142), (3, 2, 3070, 2), (2, 5, 2, 2)])
def test_space_to_depth_and_back_match_the_checker(shape):
    x = torch.arange(int(np.prod(shape)), dtype=torch.float32).reshape(shape) * 0.5 - 7
    y = rev.dt8_rev_space_to_depth(x.to(DEV))
    want = orev.space_to_depth(x.numpy(), 2)
    torch.cuda.synchronize()
    assert tuple(y.shape) == want.shape
    assert np.array_equal(y.cpu().numpy(), want)
    back = rev.dt8_rev_depth_to_space(y)
    assert np.array_equal(back.cpu().numpy(), x.numpy())
    assert np.array_equal(back.cpu().numpy(), orev.depth_to_space(want, 2))


def test_space_to_depth_at_eight_byte_offsets_and_argument_checks():
    shape = (2, 3, 4, 8)
    n = int(np.prod(shape))
    pool = torch.full((2 * n + 32,), float("nan"), device=DEV)
    xa = pool[2:2 + n].view(shape)                          # 8-byte aligned only: the 2-element path
    ya = pool[n + 7:2 * n + 7].view(2, 12, 2, 4)            # 4-byte aligned only
    x = act(shape, 2020)
    xa.copy_(x)
    rev.dt8_rev_space_to_depth(xa, ya)
    assert np.array_equal(ya.cpu().numpy(), orev.space_to_depth(x.numpy(), 2))
    assert bool(torch.isnan(pool[n + 6])) and bool(torch.isnan(pool[2 * n + 7]))
    with pytest.raises(ValueError):
        rev.dt8_rev_space_to_depth(torch.zeros(1, 1, 3, 4, device=DEV))
    with pytest.raises(dt8.DT8Error):                       # a flat side at a 4-byte-only offset
        rev.dt8_rev_space_to_depth(pool[1:1 + n].view(shape), ya)
    empty = rev.dt8_rev_space_to_depth(torch.zeros(0, 2, 4, 4, device=DEV))
    assert tuple(empty.shape) == (0, 8, 2, 2)


# ------------------------------------------------------------------------------------------------
# whole blocks
# ------------------------------------------------------------------------------------------------
def _on_cpu(fn):
    """A branch evaluated on the host whatever the device of its input, so that the CUDA path and
    the checker see identical branch outputs."""
    return lambda v: fn(v.detach().cpu()).to(v.device)


def test_block_forward_and_inverse_match_the_checker():
    shape = (3, 8, 6, 10)
    x = act(shape, 2030)
    Fb = lambda v: torch.tanh(v * 3) * 5
    Gb = lambda v: torch.sin(v) * 2
    Fn = lambda a: Fb(torch.from_numpy(a)).numpy()
    Gn = lambda a: Gb(torch.from_numpy(a)).numpy()
    y = rev.rev_block_forward(x.to(DEV), _on_cpu(Fb), _on_cpu(Gb))
    want = orev.rev_block_forward(x.numpy(), Fn, Gn)
    assert np.array_equal(y.cpu().numpy(), want)
    xr = rev.rev_block_inverse(y, _on_cpu(Fb), _on_cpu(Gb))
    assert np.array_equal(xr.cpu().numpy(), orev.rev_block_inverse(want, Fn, Gn))
    # in place
    z = x.to(DEV).clone()
    rev.rev_block_forward(z, _on_cpu(Fb), _on_cpu(Gb), out=z)
    assert np.array_equal(z.cpu().numpy(), want)
    rev.rev_block_inverse(z, _on_cpu(Fb), _on_cpu(Gb), out=z)
    assert np.array_equal(z.cpu().numpy(), xr.cpu().numpy())


def _conv_branch(c, seed):
    torch.manual_seed(seed)
    return torch.nn.Sequential(torch.nn.Conv2d(c, c, 3, padding=1), torch.nn.ReLU(),
                               torch.nn.Conv2d(c, c, 3, padding=1))


def _rel(a, b):
    a, b = a.detach().double().cpu(), b.detach().double().cpu()
    return float((a - b).norm() / (b.norm() + 1e-30))


def test_alg1_backward_matches_plain_backpropagation():
    """Alg. 1 on the GPU (binary32, library convolutions for the branches) against ordinary
    back-propagation through the stored forward pass in binary64 on the host."""
    n, c, f, t = 2, 8, 10, 12
    Fm, Gm = _conv_branch(c // 2, 1), _conv_branch(c // 2, 2)
    x = act((n, c, f, t), 2040)
    dy = act((n, c, f, t), 2041)
    y_ref, dx_ref, dwf_ref, dwg_ref = orev.rev_block_gradients(x, Fm, Gm, dy)
    Fg, Gg = _conv_branch(c // 2, 1).to(DEV), _conv_branch(c // 2, 2).to(DEV)
    y = rev.rev_block_forward(x.to(DEV), Fg, Gg)
    assert _rel(y, y_ref) < 1e-5
    xr, dx = rev.rev_block_backward(y, dy.to(DEV), Fg, Gg)
    assert _rel(xr, x) < 1e-5
    assert _rel(dx, dx_ref) < 1e-4
    for p, g in zip(Fg.parameters(), dwf_ref):
        assert _rel(p.grad, g) < 1e-4
    for p, g in zip(Gg.parameters(), dwg_ref):
        assert _rel(p.grad, g) < 1e-4
    # a second call accumulates into .grad
    rev.rev_block_backward(y, dy.to(DEV), Fg, Gg)
    assert _rel(next(Fg.parameters()).grad, 2 * dwf_ref[0]) < 1e-4


def test_rev_sequence_trains_like_the_stored_activation_network():
    """Three blocks: gradients of the reversible stack equal those of the same network run with
    ordinary autograd (binary64 on the host)."""
    n, c, f, t = 2, 6, 8, 10
    blocks = [rev.RevBlock(_conv_branch(c // 2, 10 + i), _conv_branch(c // 2, 20 + i)) for i in range(3)]
    net = rev.RevSequence(blocks).to(DEV)
    x = act((n, c, f, t), 2050).to(DEV).requires_grad_(True)
    w = act((n, c, f, t), 2051).to(DEV)
    loss = (net(x) * w).sum()
    loss.backward()
    # the same network with stored activations, binary64
    import copy
    ref = [(copy.deepcopy(b.F).double().cpu(), copy.deepcopy(b.G).double().cpu()) for b in blocks]
    xd = x.detach().double().cpu().requires_grad_(True)
    h = xd
    for Fd, Gd in ref:
        h1 = h[:, :c // 2] + Fd(h[:, c // 2:])
        h = torch.cat([h1, h[:, c // 2:] + Gd(h1)], 1)
    (h * w.double().cpu()).sum().backward()
    assert _rel(x.grad, xd.grad) < 1e-4
    for b, (Fd, Gd) in zip(blocks, ref):
        for p, q in zip(list(b.F.parameters()) + list(b.G.parameters()),
                        list(Fd.parameters()) + list(Gd.parameters())):
            assert _rel(p.grad, q.grad) < 2e-4
    # inference path keeps no graph
    with torch.no_grad():
        assert _rel(net(x), h) < 1e-5


# ------------------------------------------------------------------------------------------------
# the benchmark's shapes: the checker on sampled samples, a library identity on everything
# ------------------------------------------------------------------------------------------------
def test_benchmark_shapes_sampled_against_the_checker():
    """128 activations of the first reversible stage (48 x 80 x 200), as bench.py times them.  The
    checker follows samples 0, 77 and 127 (samples are independent); on all samples the coupling
    equals torch's element-wise add / subtract (one IEEE operation per element on both sides) and
    the rearrangement equals torch's pixel_unshuffle of the row-major reading."""
    n, c, f, t = 128, 48, 80, 200
    x = synth.normal(n * c * f * t, 1.0, 31, device=DEV).reshape(n, c, f, t)
    br = synth.normal(n * c * f * t // 2, 1.0, 32, device=DEV).reshape(n, c // 2, f, t)
    picks = [0, 77, 127]
    for which in (0, 1):
        lo, hi = (0, c // 2) if which == 0 else (c // 2, c)
        y = torch.full_like(x, float("nan"))
        rev.dt8_rev_coupling_forward(x, br, y, which)
        assert torch.equal(y[:, lo:hi], x[:, lo:hi] + br)
        want = np.full((len(picks), c, f, t), np.nan, F32)
        orev.couple_half(x[picks].cpu().numpy(), br[picks].cpu().numpy(), want, which, +1)
        assert np.array_equal(y[picks].cpu().numpy().view(np.uint32), want.view(np.uint32))
        z = torch.full_like(x, float("nan"))
        rev.dt8_rev_coupling_inverse(y, br, z, which)
        assert torch.equal(z[:, lo:hi], y[:, lo:hi] - br)
        del y, z
    del br
    for shape in ((128, 24, 80, 200), (512, 75, 20, 50)):
        n, c, f, t = shape
        a = synth.normal(n * c * f * t, 1.0, 33, device=DEV).reshape(shape)
        d = rev.dt8_rev_space_to_depth(a)
        assert torch.equal(d, torch.nn.functional.pixel_unshuffle(a, 2))
        for k in (0, n // 2 + 1, n - 1):
            assert np.array_equal(d[k:k + 1].cpu().numpy(), orev.space_to_depth(a[k:k + 1].cpu().numpy(), 2))
        assert torch.equal(rev.dt8_rev_depth_to_space(d), a)
        del a, d

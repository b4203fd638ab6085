"""rev oracle -- TEST INFRASTRUCTURE, NOT THE PRODUCT.

numpy-facing wrapper around ``rev_oracle.c``: the additive coupling of a reversible residual
block (Eq. revnet4), its inverse (Eq. revnet5) and the invertible down-sampling of Eq. revnet6
(Section III-B of the paper), plus the whole-block forms that take the residual branches F and G
as Python callables, and the gradients Alg. 1 must produce, obtained the plain way (ordinary
back-propagation through the stored forward pass, in binary64).

Only tests, the smoke check and the benchmark's cpu-baseline leg may import this module; the CUDA
library and its Python binding never do, and this module imports nothing from them.

Parity unpinned: the order of the r*r*C output channels of the down-sampling against the authors'
implementation (the paper gives the shape only); everything else is pinned by the
``-m "not gpu"`` tests.
"""
from __future__ import annotations

import ctypes
import os
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "rev_oracle.c")

_lock = threading.Lock()
_lib = None


def build(force: bool = False) -> str:
    from . import build_source
    return build_source(_SRC, "librev_oracle.so", "REV_ORACLE_SOURCE", force)


def _load():
    global _lib
    with _lock:
        if _lib is None:
            lib = ctypes.CDLL(build())
            c = ctypes
            fp, i64 = c.POINTER(c.c_float), c.c_int64
            lib.revo_couple_half.argtypes = [fp, fp, fp, i64, i64, c.c_int, c.c_int]
            lib.revo_space_to_depth.argtypes = [fp, i64, i64, i64, i64, c.c_int, fp]
            lib.revo_depth_to_space.argtypes = [fp, i64, i64, i64, i64, c.c_int, fp]
            _lib = lib
    return _lib


def _f32(a, name):
    if not (isinstance(a, np.ndarray) and a.dtype == np.float32 and a.flags.c_contiguous):
        raise TypeError(f"{name}: need a C-contiguous float32 ndarray")
    return a.ctypes.data_as(ctypes.POINTER(ctypes.c_float))


def couple_half(inp: np.ndarray, t: np.ndarray, out: np.ndarray, which: int, sign: int) -> None:
    """out[:, half `which`] = inp[:, half `which`] + sign * t, for N x C x F x T arrays `inp`, `out`
    and the branch output `t` of shape N x C/2 x F x T; the other half of `out` is left alone."""
    if inp.ndim != 4 or inp.shape[1] % 2 or out.shape != inp.shape:
        raise ValueError("N x C x F x T arrays with an even number of channels are required")
    n, ch, f, tt = inp.shape
    if t.shape != (n, ch // 2, f, tt):
        raise ValueError("t: N x C/2 x F x T required")
    rc = _load().revo_couple_half(_f32(inp, "inp"), _f32(t, "t"), _f32(out, "out"), n,
                                  (ch // 2) * f * tt, which, sign)
    if rc:
        raise ValueError("rev oracle couple_half: bad arguments")


def rev_block_forward(x: np.ndarray, F, G) -> np.ndarray:
    """Eq. revnet4: y1 = x1 + F(x2); y2 = x2 + G(y1), with x1 / x2 the two channel halves."""
    c = x.shape[1] // 2
    y = np.empty_like(x)
    f_out = np.ascontiguousarray(F(np.ascontiguousarray(x[:, c:])), np.float32)
    couple_half(x, f_out, y, 0, +1)
    g_out = np.ascontiguousarray(G(np.ascontiguousarray(y[:, :c])), np.float32)
    couple_half(x, g_out, y, 1, +1)
    return y


def rev_block_inverse(y: np.ndarray, F, G) -> np.ndarray:
    """Eq. revnet5: z1 = y1; x2 = y2 - G(z1); x1 = z1 - F(x2)."""
    c = y.shape[1] // 2
    x = np.empty_like(y)
    g_out = np.ascontiguousarray(G(np.ascontiguousarray(y[:, :c])), np.float32)
    couple_half(y, g_out, x, 1, -1)
    f_out = np.ascontiguousarray(F(np.ascontiguousarray(x[:, c:])), np.float32)
    couple_half(y, f_out, x, 0, -1)
    return x


def space_to_depth(x: np.ndarray, r: int = 2) -> np.ndarray:
    """Eq. revnet6: N x C x F x T -> N x r*r*C x F/r x T/r."""
    n, c, f, t = x.shape
    if f % r or t % r:
        raise ValueError("F and T must be multiples of r")
    y = np.empty((n, c * r * r, f // r, t // r), np.float32)
    rc = _load().revo_space_to_depth(_f32(x, "x"), n, c, f, t, r, _f32(y, "y"))
    if rc:
        raise ValueError("rev oracle space_to_depth: bad arguments")
    return y


def depth_to_space(y: np.ndarray, r: int = 2) -> np.ndarray:
    """The inverse of Eq. revnet6: N x r*r*C x Fo x To -> N x C x Fo*r x To*r."""
    n, cc, fo, to = y.shape
    if cc % (r * r):
        raise ValueError("the channel count must be a multiple of r*r")
    x = np.empty((n, cc // (r * r), fo * r, to * r), np.float32)
    rc = _load().revo_depth_to_space(_f32(y, "y"), n, cc // (r * r), fo, to, r, _f32(x, "x"))
    if rc:
        raise ValueError("rev oracle depth_to_space: bad arguments")
    return x


def rev_block_gradients(x, F, G, dy):
    """What Alg. 1 must return, obtained the plain way: the forward pass of Eq. revnet4 is run
    with every activation stored, in binary64, and ordinary back-propagation gives dL/dx and the
    gradients of the branches' parameters for the output gradient dy.

    x, dy: torch tensors N x C x F x T; F, G: torch modules (their parameters are read, not
    changed).  Returns (y, dx, [dL/dw for w in F.parameters()], [... G.parameters()]), binary64."""
    import copy

    import torch
    Fd, Gd = copy.deepcopy(F).double(), copy.deepcopy(G).double()
    xd = x.detach().double().cpu().requires_grad_(True)
    Fd, Gd = Fd.cpu(), Gd.cpu()
    c = xd.shape[1] // 2
    x1, x2 = xd[:, :c], xd[:, c:]
    y1 = x1 + Fd(x2)
    y2 = x2 + Gd(y1)
    y = torch.cat([y1, y2], dim=1)
    params = list(Fd.parameters()) + list(Gd.parameters())
    grads = torch.autograd.grad(y, [xd] + params, dy.detach().double().cpu(), allow_unused=True)
    nf = len(list(Fd.parameters()))
    return y.detach(), grads[0], list(grads[1:1 + nf]), list(grads[1 + nf:])

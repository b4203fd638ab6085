"""Reversible-network memory kernels (Section III-B of the paper): Python binding.

``dt8_rev_*`` are thin wrappers of the C ABI in ``include/dt8_rev.h`` (argument marshalling only).
On top of them sit the whole-block forms, which call the residual branches F and G -- any
callables / ``torch.nn.Module``s, supplied by the caller -- and run every element-wise step of
Eq. revnet4, Eq. revnet5 and Alg. 1 in the CUDA library:

    rev_block_forward(x, F, G)         y1 = x1 + F(x2);  y2 = x2 + G(y1)
    rev_block_inverse(y, F, G)         x2 = y2 - G(y1);  x1 = y1 - F(x2)
    rev_block_backward(y, dy, F, G)    Alg. 1: recovers x, returns dL/dx, accumulates dL/dw
    RevSequence(blocks)                a stack of blocks that keeps no activation between them

There is no CPU implementation behind these functions.
"""
from __future__ import annotations

import ctypes
from typing import Optional, Sequence

import torch

from . import DT8Error, DT8_OK, _on_device, _stream_ptr, load_library

__all__ = ["dt8_rev_coupling_forward", "dt8_rev_coupling_inverse", "dt8_rev_space_to_depth",
           "dt8_rev_depth_to_space", "rev_block_forward", "rev_block_inverse", "rev_block_backward",
           "RevBlock", "RevSequence"]

REV_EXPORTS = ("dt8_rev_coupling_forward", "dt8_rev_coupling_inverse", "dt8_rev_space_to_depth",
               "dt8_rev_depth_to_space")
_bound = False


def _lib():
    global _bound
    lib = load_library()
    if not _bound:
        vp, i64, i32 = ctypes.c_void_p, ctypes.c_int64, ctypes.c_int
        lib.dt8_rev_coupling_forward.argtypes = [vp, vp, vp, i64, i64, i32, vp]
        lib.dt8_rev_coupling_inverse.argtypes = [vp, vp, vp, i64, i64, i32, vp]
        lib.dt8_rev_space_to_depth.argtypes = [vp, i64, i64, i64, i64, vp, vp]
        lib.dt8_rev_depth_to_space.argtypes = [vp, i64, i64, i64, i64, vp, vp]
        for name in REV_EXPORTS:
            getattr(lib, name).restype = i32
        _bound = True
    return lib


def _act(t: torch.Tensor, name: str) -> int:
    if not (isinstance(t, torch.Tensor) and t.is_cuda and t.is_contiguous() and t.dtype == torch.float32):
        raise TypeError(f"{name}: need a contiguous float32 CUDA tensor")
    return t.data_ptr()


def _check(status: int, where: str) -> None:
    if status != DT8_OK:
        raise DT8Error(status, where)


def _couple(fn_name: str, a: torch.Tensor, t: torch.Tensor, out: torch.Tensor, which: int, stream) -> None:
    if a.dim() < 2 or a.shape[1] % 2:
        raise ValueError(f"{fn_name}: N x C x ... activation with an even number of channels required")
    n = a.shape[0]
    half = 1
    for d in a.shape[1:]:
        half *= int(d)
    half //= 2
    if out.shape != a.shape or t.numel() != n * half or t.device != a.device or out.device != a.device:
        raise ValueError(f"{fn_name}: out must have the activation's shape and t half of its elements, "
                         "all on one device")
    with _on_device(a.device):
        st = getattr(_lib(), fn_name)(_act(a, "activation"), _act(t, "t"), _act(out, "out"), n, half,
                                      int(which), _stream_ptr(stream, a.device))
    _check(st, fn_name)


def dt8_rev_coupling_forward(x, t, y, which: int, stream=None) -> None:
    """y[:, half `which`] = x[:, half `which`] + t (Eq. revnet4); y may be x."""
    _couple("dt8_rev_coupling_forward", x, t, y, which, stream)


def dt8_rev_coupling_inverse(y, t, x, which: int, stream=None) -> None:
    """x[:, half `which`] = y[:, half `which`] - t (Eq. revnet5); x may be y."""
    _couple("dt8_rev_coupling_inverse", y, t, x, which, stream)


def dt8_rev_space_to_depth(x: torch.Tensor, out: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
    """Eq. revnet6 with r = 2: N x C x F x T -> N x 4C x F/2 x T/2."""
    if x.dim() != 4 or x.shape[2] % 2 or x.shape[3] % 2:
        raise ValueError("dt8_rev_space_to_depth: N x C x F x T with even F and T required")
    n, c, f, t = x.shape
    if out is None:
        out = torch.empty((n, 4 * c, f // 2, t // 2), dtype=torch.float32, device=x.device)
    if out.numel() != x.numel() or out.device != x.device:
        raise ValueError("dt8_rev_space_to_depth: out must hold as many elements as x, on its device")
    with _on_device(x.device):
        st = _lib().dt8_rev_space_to_depth(_act(x, "x"), n, c, f, t, _act(out, "out"),
                                           _stream_ptr(stream, x.device))
    _check(st, "dt8_rev_space_to_depth")
    return out


def dt8_rev_depth_to_space(y: torch.Tensor, out: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
    """The inverse of Eq. revnet6 with r = 2: N x 4C x Fo x To -> N x C x 2Fo x 2To."""
    if y.dim() != 4 or y.shape[1] % 4:
        raise ValueError("dt8_rev_depth_to_space: N x 4C x Fo x To required")
    n, c4, fo, to = y.shape
    if out is None:
        out = torch.empty((n, c4 // 4, 2 * fo, 2 * to), dtype=torch.float32, device=y.device)
    if out.numel() != y.numel() or out.device != y.device:
        raise ValueError("dt8_rev_depth_to_space: out must hold as many elements as y, on its device")
    with _on_device(y.device):
        st = _lib().dt8_rev_depth_to_space(_act(y, "y"), n, c4 // 4, fo, to, _act(out, "out"),
                                           _stream_ptr(stream, y.device))
    _check(st, "dt8_rev_depth_to_space")
    return out


# -----------------------------------------------------------------------------------------------
# whole blocks: the branches are the caller's, every coupling step is a library kernel
# -----------------------------------------------------------------------------------------------
def _halves(a: torch.Tensor):
    c = a.shape[1] // 2
    return a[:, :c], a[:, c:]


def _branch(fn, v: torch.Tensor) -> torch.Tensor:
    out = fn(v)
    if out.shape != v.shape:
        raise ValueError("a residual branch must keep the shape of its input (stride 1, Section III-B)")
    return out


def rev_block_forward(x: torch.Tensor, F, G, out: Optional[torch.Tensor] = None) -> torch.Tensor:
    """Eq. revnet4 on an N x C x F x T activation whose channel halves are x1, x2.  No graph is
    recorded; out may be x (in place)."""
    y = torch.empty_like(x) if out is None else out
    with torch.no_grad():
        _, x2 = _halves(x)
        dt8_rev_coupling_forward(x, _branch(F, x2).contiguous(), y, 0)
        y1, _ = _halves(y)
        dt8_rev_coupling_forward(x, _branch(G, y1).contiguous(), y, 1)
    return y


def rev_block_inverse(y: torch.Tensor, F, G, out: Optional[torch.Tensor] = None) -> torch.Tensor:
    """Eq. revnet5: the input of the block from its output; out may be y (in place)."""
    x = torch.empty_like(y) if out is None else out
    with torch.no_grad():
        z1, _ = _halves(y)
        dt8_rev_coupling_inverse(y, _branch(G, z1).contiguous(), x, 1)     # x2 = y2 - G(z1)
        _, x2 = _halves(x)
        dt8_rev_coupling_inverse(y, _branch(F, x2).contiguous(), x, 0)     # x1 = z1 - F(x2)
    return x


def _params(fn) -> list:
    return [p for p in fn.parameters() if p.requires_grad] if isinstance(fn, torch.nn.Module) else []


def _accumulate(params: Sequence[torch.Tensor], grads: Sequence[Optional[torch.Tensor]]) -> None:
    for p, g in zip(params, grads):
        if g is None:
            continue
        if p.grad is None:
            p.grad = g.detach().clone()
        else:
            p.grad.add_(g)


def rev_block_backward(y: torch.Tensor, dy: torch.Tensor, F, G, x_out: Optional[torch.Tensor] = None,
                       dx_out: Optional[torch.Tensor] = None):
    """Alg. 1.  Given the block's output y and dL/dy, recovers the input x, returns dL/dx and
    adds the gradients of the branches' parameters to their .grad.  The branches are re-run once
    each with a graph (that is the recomputation the method trades for memory); their
    vector-Jacobian products come from torch.autograd, the sums and differences from the library.
    x_out may be y and dx_out may be dy (in place)."""
    x = torch.empty_like(y) if x_out is None else x_out
    dx = torch.empty_like(dy) if dx_out is None else dx_out
    pF, pG = _params(F), _params(G)
    _, dy2 = _halves(dy)
    # z1 = y1;  x2 = y2 - G(z1)
    z1 = _halves(y)[0].detach().requires_grad_(True)
    with torch.enable_grad():
        g = _branch(G, z1)
    dt8_rev_coupling_inverse(y, g.detach().contiguous(), x, 1)
    # dL/dz1 = dL/dy1 + (dG/dz1)^T dL/dy2;  dL/dwG = (dG/dwG)^T dL/dy2
    grads = torch.autograd.grad(g, [z1] + pG, dy2, allow_unused=True)
    del g
    dt8_rev_coupling_forward(dy, grads[0].contiguous(), dx, 0)
    _accumulate(pG, grads[1:])
    # x1 = z1 - F(x2)
    x2 = _halves(x)[1].detach().requires_grad_(True)
    with torch.enable_grad():
        f = _branch(F, x2)
    dt8_rev_coupling_inverse(y, f.detach().contiguous(), x, 0)
    # dL/dx2 = dL/dy2 + (dF/dx2)^T dL/dz1;  dL/dx1 = dL/dz1;  dL/dwF = (dF/dwF)^T dL/dz1
    dz1 = _halves(dx)[0]
    grads = torch.autograd.grad(f, [x2] + pF, dz1, allow_unused=True)
    del f
    dt8_rev_coupling_forward(dy, grads[0].contiguous(), dx, 1)
    _accumulate(pF, grads[1:])
    return x, dx


class RevBlock(torch.nn.Module):
    """A reversible residual block (Section III-B): two residual branches of C/2 channels."""

    def __init__(self, F: torch.nn.Module, G: torch.nn.Module):
        super().__init__()
        self.F, self.G = F, G

    def forward(self, x: torch.Tensor) -> torch.Tensor:
        return rev_block_forward(x, self.F, self.G)


class _RevSequenceFn(torch.autograd.Function):
    """Forward through all blocks keeping only the last output; backward walks the blocks in
    reverse with Alg. 1, recovering each block's input from its output in the same buffer."""

    @staticmethod
    def forward(ctx, x, blocks, *params):
        ctx.blocks = blocks
        y = x.detach().clone()
        for blk in blocks:
            rev_block_forward(y, blk.F, blk.G, out=y)
        ctx.save_for_backward(y)
        return y

    @staticmethod
    def backward(ctx, dy):
        (y,) = ctx.saved_tensors
        cur = y.detach().clone()          # the saved output itself must stay intact for autograd
        dcur = dy.contiguous().clone()
        for blk in reversed(ctx.blocks):
            rev_block_backward(cur, dcur, blk.F, blk.G, x_out=cur, dx_out=dcur)
        return (dcur, None) + tuple(None for _ in ctx.needs_input_grad[2:])


class RevSequence(torch.nn.Module):
    """A stack of RevBlocks trained without storing the activations between them: memory for
    activations does not grow with the number of blocks (Section III-B).  Parameter gradients
    are accumulated into .grad during the backward pass, as torch's own backward does.  The
    branches are run twice per training step (forward, and once more in Alg. 1), so layers with
    running statistics see every batch twice."""

    def __init__(self, blocks: Sequence[RevBlock]):
        super().__init__()
        self.blocks = torch.nn.ModuleList(blocks)

    def forward(self, x: torch.Tensor) -> torch.Tensor:
        params = [p for p in self.parameters() if p.requires_grad]
        if torch.is_grad_enabled() and (x.requires_grad or params):
            return _RevSequenceFn.apply(x, list(self.blocks), *params)
        y = x.detach().clone()
        for blk in self.blocks:
            rev_block_forward(y, blk.F, blk.G, out=y)
        return y

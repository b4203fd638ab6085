"""dt8: fused 8-bit optimizer step over the dynamic-tree 8-bit data type, for NVIDIA B200.

Thin Python binding of the C ABI in ``include/dt8.h`` (same names, argument marshalling
only).  Every step of the method runs in the CUDA library ``libdt8.so``; PyTorch is used for
device memory and streams.  There is no CPU implementation behind these functions: if the
library is missing or no CUDA device is present, the calls raise.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional, Sequence

import numpy as np
import torch

__all__ = [
    "DT8Error", "lib_path", "load_library", "num_blocks",
    "dt8_codebook", "dt8_state_bytes", "optimizer_state_bytes", "dt8_selfcheck_encode_host", "dt8_selfcheck_divide", "dt8_selfcheck_divide_const", "dt8_selfcheck_reciprocal", "dt8_selfcheck_root", "dt8_init",
    "dt8_quantize_blockwise",
    "dt8_dequantize_blockwise", "dt8_sgd_step", "dt8_adam_step", "dt8_sgd_step_multi",
    "dt8_adam_step_multi", "new_state", "shard_blocks", "PreparedTensorList",
    "DT8_F32", "DT8_BF16", "DT8_ADAM_BIAS_CORRECTION", "DT8_ADAM_DECOUPLED_WD", "DEFAULT_ADAM_FLAGS",
    "BLOCK_SIZES",
]

DT8_OK, DT8_ERR_INVALID_ARG, DT8_ERR_UNSUPPORTED, DT8_ERR_ALIGNMENT, DT8_ERR_CUDA = range(5)
DT8_F32, DT8_BF16 = 0, 1
DT8_ADAM_BIAS_CORRECTION, DT8_ADAM_DECOUPLED_WD = 1, 2
DEFAULT_ADAM_FLAGS = DT8_ADAM_BIAS_CORRECTION | DT8_ADAM_DECOUPLED_WD
BLOCK_SIZES = (256, 512, 1024, 2048, 4096)

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_HERE, "libdt8.so")
_lib = None

EXPORTS = (
    "dt8_status_string", "dt8_last_cuda_error", "dt8_codebook", "dt8_state_bytes",
    "dt8_selfcheck_encode_host",
    "dt8_selfcheck_divide", "dt8_selfcheck_divide_const", "dt8_selfcheck_reciprocal", "dt8_selfcheck_root", "dt8_init",
    "dt8_quantize_blockwise",
    "dt8_dequantize_blockwise", "dt8_sgd_step",
    "dt8_adam_step", "dt8_sgd_step_multi", "dt8_adam_step_multi",
    "dt8_sgd_step_ex", "dt8_adam_step_ex", "dt8_sgd_step_multi_ex", "dt8_adam_step_multi_ex",
    "dt8_selfcheck_table_extents", "dt8_selfcheck_layout_fits",
)


class DT8Error(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        msg = load_library().dt8_status_string(status).decode()
        if status == DT8_ERR_CUDA:
            msg += " [cudaError %d]" % load_library().dt8_last_cuda_error()
        super().__init__(f"{where}: {msg}")


def lib_path() -> str:
    return _LIB_PATH


def load_library() -> ctypes.CDLL:
    """Loads libdt8.so (built in-tree by ``paper_2412_01195_b200.build``); raises if absent."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(_LIB_PATH):
        raise RuntimeError(
            f"{_LIB_PATH} is missing: build it with `python -m paper_2412_01195_b200.build` "
            "(there is no fallback implementation)")
    lib = ctypes.CDLL(_LIB_PATH)
    c = ctypes
    vp, i64, f32, i32, u32 = c.c_void_p, c.c_int64, c.c_float, c.c_int, c.c_uint32
    lib.dt8_status_string.restype = c.c_char_p
    lib.dt8_status_string.argtypes = [i32]
    lib.dt8_last_cuda_error.restype = i32
    lib.dt8_codebook.argtypes = [i32, vp]
    lib.dt8_state_bytes.argtypes = [i64, i32]
    lib.dt8_state_bytes.restype = i64
    lib.dt8_selfcheck_encode_host.argtypes = [i32, vp, i64, vp]
    lib.dt8_selfcheck_divide.argtypes = [vp, vp, i64, vp, vp]
    lib.dt8_selfcheck_divide_const.argtypes = [vp, f32, i64, vp, vp]
    lib.dt8_selfcheck_reciprocal.argtypes = [vp, i64, vp, vp]
    lib.dt8_selfcheck_root.argtypes = [vp, i64, vp, vp]
    lib.dt8_selfcheck_table_extents.argtypes = [vp, vp, vp, vp]
    lib.dt8_selfcheck_layout_fits.argtypes = [u32, i32, u32, i32]
    lib.dt8_init.argtypes = []
    lib.dt8_quantize_blockwise.argtypes = [vp, i64, i32, i32, vp, vp, vp]
    lib.dt8_dequantize_blockwise.argtypes = [vp, vp, i64, i32, i32, vp, vp]
    lib.dt8_sgd_step.argtypes = [vp, vp, i32, vp, vp, i64, f32, f32, f32, i64, i32, vp]
    lib.dt8_adam_step.argtypes = [vp, vp, i32, vp, vp, vp, vp, i64, f32, f32, f32, f32, f32, i64, i32,
                                  u32, vp]
    lib.dt8_sgd_step_multi.argtypes = [i32, vp, vp, i32, vp, vp, vp, f32, f32, f32, i64, i32, vp]
    lib.dt8_adam_step_multi.argtypes = [i32, vp, vp, i32, vp, vp, vp, vp, vp, f32, f32, f32, f32, f32,
                                        i64, i32, u32, vp]
    lib.dt8_sgd_step_ex.argtypes = [vp, i32, vp, i32, vp, vp, i64, f32, f32, f32, i64, i32, vp]
    lib.dt8_adam_step_ex.argtypes = [vp, i32, vp, i32, vp, vp, vp, vp, i64, f32, f32, f32, f32, f32, i64,
                                     i32, u32, vp]
    lib.dt8_sgd_step_multi_ex.argtypes = [i32, vp, i32, vp, i32, vp, vp, vp, f32, f32, f32, i64, i32, vp]
    lib.dt8_adam_step_multi_ex.argtypes = [i32, vp, i32, vp, i32, vp, vp, vp, vp, vp, f32, f32, f32, f32,
                                           f32, i64, i32, u32, vp]
    for name in EXPORTS:
        getattr(lib, name).restype = getattr(lib, name).restype or i32
    _lib = lib
    return lib


def _check(status: int, where: str) -> None:
    if status != DT8_OK:
        raise DT8Error(status, where)


def num_blocks(n: int, block_size: int) -> int:
    return (n + block_size - 1) // block_size


class _on_device:
    """`with torch.cuda.device(d)` only when d is not already the current device (the context
    manager costs several microseconds per call, as much as a small launch)."""

    def __init__(self, device):
        idx = device.index if device.index is not None else torch.cuda.current_device()
        self._guard = None if idx == torch.cuda.current_device() else torch.cuda.device(idx)

    def __enter__(self):
        if self._guard is not None:
            self._guard.__enter__()

    def __exit__(self, *exc):
        if self._guard is not None:
            self._guard.__exit__(*exc)
        return False


def _stream_ptr(stream: Optional[torch.cuda.Stream], device) -> int:
    s = stream if stream is not None else torch.cuda.current_stream(device)
    return s.cuda_stream


def _dev_tensor(t: torch.Tensor, dtype, name: str) -> int:
    if not (isinstance(t, torch.Tensor) and t.is_cuda and t.is_contiguous() and t.dtype == dtype):
        raise TypeError(f"{name}: need a contiguous CUDA tensor of dtype {dtype}")
    return t.data_ptr()


def _check_layout(where: str, n: int, block_size: int, device, by_elements: dict, by_blocks: dict) -> None:
    """The C ABI takes n and block_size on trust; the tensors' own sizes are known here.  A state
    built for another block size, a gradient of another length or a tensor on another device would
    make the kernel read or write outside an allocation, so each is refused before the call."""
    if block_size not in BLOCK_SIZES:
        raise ValueError(f"{where}: block_size must be one of {BLOCK_SIZES}")
    nb = num_blocks(n, block_size)
    for name, t in by_elements.items():
        if t.numel() != n:
            raise ValueError(f"{where}: {name} holds {t.numel()} elements, expected {n}")
    for name, t in by_blocks.items():
        if t.numel() != nb:
            raise ValueError(f"{where}: {name} holds {t.numel()} block maxima, expected {nb} "
                             f"(= ceil({n} / {block_size}))")
    for name, t in {**by_elements, **by_blocks}.items():
        if t.device != device:
            raise ValueError(f"{where}: {name} is on {t.device}, expected {device}")


def _grad_ptr(g: torch.Tensor, name: str = "g"):
    """(device pointer, dt8_dtype) of a gradient or parameter tensor: float32 or bfloat16."""
    if not (isinstance(g, torch.Tensor) and g.is_cuda and g.is_contiguous()):
        raise TypeError(f"{name}: need a contiguous CUDA tensor")
    if g.dtype == torch.float32:
        return g.data_ptr(), DT8_F32
    if g.dtype == torch.bfloat16:
        return g.data_ptr(), DT8_BF16
    raise TypeError(f"{name}: float32 or bfloat16")


# -----------------------------------------------------------------------------------------------
# host-only entry points
# -----------------------------------------------------------------------------------------------
def dt8_codebook(is_signed: bool) -> np.ndarray:
    """The 256 ascending values of the data type (host, no GPU needed)."""
    out = np.empty(256, np.float32)
    _check(load_library().dt8_codebook(int(bool(is_signed)), out.ctypes.data), "dt8_codebook")
    return out


def dt8_state_bytes(n: int, block_size: int = 2048) -> int:
    """Bytes of one 8-bit state of n elements (codes + one fp32 maximum per block)."""
    b = load_library().dt8_state_bytes(n, block_size)
    if b < 0:
        raise ValueError("dt8_state_bytes: n >= 0 and a supported block size are required")
    return int(b)


def optimizer_state_bytes(sizes: Sequence[int], states_per_weight: int, block_size: int = 2048):
    """(32-bit bytes, 8-bit bytes) of the optimizer state of a tensor list: SGD with momentum
    keeps one state per weight, Adam two; every tensor is chunked on its own."""
    full = 4 * states_per_weight * sum(int(n) for n in sizes)
    small = states_per_weight * sum(dt8_state_bytes(int(n), block_size) for n in sizes)
    return full, small


def dt8_selfcheck_encode_host(is_signed: bool, v: np.ndarray) -> np.ndarray:
    """Diagnostic: the kernels' table-driven nearest-code search run on the host."""
    v = np.ascontiguousarray(v, np.float32).ravel()
    out = np.empty(v.size, np.uint8)
    _check(load_library().dt8_selfcheck_encode_host(int(bool(is_signed)), v.ctypes.data, v.size,
                                                    out.ctypes.data), "dt8_selfcheck_encode_host")
    return out


# -----------------------------------------------------------------------------------------------
# device entry points
# -----------------------------------------------------------------------------------------------
def dt8_init(device=None) -> None:
    with torch.cuda.device(device if device is not None else torch.cuda.current_device()):
        _check(load_library().dt8_init(), "dt8_init")


def dt8_selfcheck_divide(s: torch.Tensor, N: torch.Tensor, out: Optional[torch.Tensor] = None,
                         stream=None) -> torch.Tensor:
    """Diagnostic: the kernels' normalising division applied to operand pairs (s_i, N_i)."""
    if out is None:
        out = torch.empty_like(s)
    with _on_device(s.device):
        st = load_library().dt8_selfcheck_divide(
            _dev_tensor(s, torch.float32, "s"), _dev_tensor(N, torch.float32, "N"), s.numel(),
            _dev_tensor(out, torch.float32, "out"), _stream_ptr(stream, s.device))
    _check(st, "dt8_selfcheck_divide")
    return out


def dt8_selfcheck_reciprocal(N: torch.Tensor, out: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
    """Diagnostic: the reciprocal of N_i the normalising division starts from (0 where it takes
    the IEEE division)."""
    if out is None:
        out = torch.empty_like(N)
    with _on_device(N.device):
        st = load_library().dt8_selfcheck_reciprocal(
            _dev_tensor(N, torch.float32, "N"), N.numel(), _dev_tensor(out, torch.float32, "out"),
            _stream_ptr(stream, N.device))
    _check(st, "dt8_selfcheck_reciprocal")
    return out


def dt8_selfcheck_root(x: torch.Tensor, out: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
    """Diagnostic: the square root of the fast IEEE Adam parameter update (0 outside its range)."""
    if out is None:
        out = torch.empty_like(x)
    with _on_device(x.device):
        st = load_library().dt8_selfcheck_root(
            _dev_tensor(x, torch.float32, "x"), x.numel(), _dev_tensor(out, torch.float32, "out"),
            _stream_ptr(stream, x.device))
    _check(st, "dt8_selfcheck_root")
    return out


def dt8_selfcheck_divide_const(s: torch.Tensor, d: float, out: Optional[torch.Tensor] = None,
                               stream=None) -> torch.Tensor:
    """Diagnostic: the constant-divisor division of the IEEE Adam update applied to (s_i, d)."""
    if out is None:
        out = torch.empty_like(s)
    with _on_device(s.device):
        st = load_library().dt8_selfcheck_divide_const(
            _dev_tensor(s, torch.float32, "s"), float(d), s.numel(),
            _dev_tensor(out, torch.float32, "out"), _stream_ptr(stream, s.device))
    _check(st, "dt8_selfcheck_divide_const")
    return out


def new_state(n: int, block_size: int, signed: bool, device) -> tuple:
    """Zero state: canonical zero codes and absmax 0."""
    codes = torch.full((n,), 127 if signed else 0, dtype=torch.uint8, device=device)
    absmax = torch.zeros(num_blocks(n, block_size), dtype=torch.float32, device=device)
    return codes, absmax


def dt8_quantize_blockwise(x: torch.Tensor, block_size: int, is_signed: bool,
                           codes: Optional[torch.Tensor] = None, absmax: Optional[torch.Tensor] = None,
                           stream=None):
    n = x.numel()
    if block_size not in BLOCK_SIZES:
        raise ValueError(f"dt8_quantize_blockwise: block_size must be one of {BLOCK_SIZES}")
    if codes is None:
        codes = torch.empty(n, dtype=torch.uint8, device=x.device)
    if absmax is None:
        absmax = torch.empty(num_blocks(n, block_size), dtype=torch.float32, device=x.device)
    _check_layout("dt8_quantize_blockwise", n, block_size, x.device, {"codes": codes}, {"absmax": absmax})
    with _on_device(x.device):
        st = load_library().dt8_quantize_blockwise(
            _dev_tensor(x, torch.float32, "x"), n, block_size, int(bool(is_signed)),
            _dev_tensor(codes, torch.uint8, "codes"), _dev_tensor(absmax, torch.float32, "absmax"),
            _stream_ptr(stream, x.device))
    _check(st, "dt8_quantize_blockwise")
    return codes, absmax


def dt8_dequantize_blockwise(codes: torch.Tensor, absmax: torch.Tensor, block_size: int,
                             is_signed: bool, out: Optional[torch.Tensor] = None, stream=None):
    n = codes.numel()
    if out is None:
        out = torch.empty(n, dtype=torch.float32, device=codes.device)
    _check_layout("dt8_dequantize_blockwise", n, block_size, codes.device, {"out": out}, {"absmax": absmax})
    with _on_device(codes.device):
        st = load_library().dt8_dequantize_blockwise(
            _dev_tensor(codes, torch.uint8, "codes"), _dev_tensor(absmax, torch.float32, "absmax"), n,
            block_size, int(bool(is_signed)), _dev_tensor(out, torch.float32, "out"),
            _stream_ptr(stream, codes.device))
    _check(st, "dt8_dequantize_blockwise")
    return out


def dt8_sgd_step(p, g, m_codes, m_absmax, lr, momentum, weight_decay, step, block_size=2048,
                 stream=None) -> None:
    _check_layout("dt8_sgd_step", p.numel(), block_size, p.device, {"g": g, "m_codes": m_codes},
                  {"m_absmax": m_absmax})
    gp, gd = _grad_ptr(g)
    pp, pd = _grad_ptr(p, "p")
    with _on_device(p.device):
        st = load_library().dt8_sgd_step_ex(
            pp, pd, gp, gd, _dev_tensor(m_codes, torch.uint8, "m_codes"),
            _dev_tensor(m_absmax, torch.float32, "m_absmax"), p.numel(), lr, momentum, weight_decay,
            step, block_size, _stream_ptr(stream, p.device))
    _check(st, "dt8_sgd_step")


def dt8_adam_step(p, g, m_codes, m_absmax, r_codes, r_absmax, lr, beta1, beta2, eps, weight_decay,
                  step, block_size=2048, flags=DEFAULT_ADAM_FLAGS, stream=None) -> None:
    _check_layout("dt8_adam_step", p.numel(), block_size, p.device,
                  {"g": g, "m_codes": m_codes, "r_codes": r_codes},
                  {"m_absmax": m_absmax, "r_absmax": r_absmax})
    gp, gd = _grad_ptr(g)
    pp, pd = _grad_ptr(p, "p")
    with _on_device(p.device):
        st = load_library().dt8_adam_step_ex(
            pp, pd, gp, gd, _dev_tensor(m_codes, torch.uint8, "m_codes"),
            _dev_tensor(m_absmax, torch.float32, "m_absmax"), _dev_tensor(r_codes, torch.uint8, "r_codes"),
            _dev_tensor(r_absmax, torch.float32, "r_absmax"), p.numel(), lr, beta1, beta2, eps,
            weight_decay, step, block_size, flags, _stream_ptr(stream, p.device))
    _check(st, "dt8_adam_step")


class _PtrList:
    """Host arrays of device pointers / sizes for the pointer-list entry points."""

    def __init__(self, tensors: Sequence[torch.Tensor], dtype, name: str):
        self.arr = (ctypes.c_void_p * len(tensors))(*[_dev_tensor(t, dtype, name) for t in tensors])

    @property
    def ptr(self):
        return ctypes.cast(self.arr, ctypes.c_void_p)


def _check_list_layout(where, block_size, ps, gs, m_codes, m_absmax, r_codes=None, r_absmax=None):
    lists = {"g": gs, "m_codes": m_codes, "m_absmax": m_absmax}
    if r_codes is not None:
        lists["r_codes"], lists["r_absmax"] = r_codes, r_absmax
    for name, lst in lists.items():
        if len(lst) != len(ps):
            raise ValueError(f"{where}: {name} lists {len(lst)} tensors, expected {len(ps)}")
    dev = ps[0].device if len(ps) else None
    for i, p in enumerate(ps):
        by_el = {f"g[{i}]": gs[i], f"m_codes[{i}]": m_codes[i]}
        by_bl = {f"m_absmax[{i}]": m_absmax[i]}
        if r_codes is not None:
            by_el[f"r_codes[{i}]"] = r_codes[i]
            by_bl[f"r_absmax[{i}]"] = r_absmax[i]
        if p.device != dev:
            raise ValueError(f"{where}: p[{i}] is on {p.device}, expected {dev}")
        _check_layout(where, p.numel(), block_size, dev, by_el, by_bl)


class _TypedPtrList:
    """Host array of device pointers of tensors that share one of the two element types."""

    def __init__(self, tensors: Sequence[torch.Tensor], name: str):
        dt = tensors[0].dtype
        if any(t.dtype != dt for t in tensors):
            raise TypeError(f"all {name} tensors of one call share a dtype")
        self.dtype = _grad_ptr(tensors[0], name)[1]
        self.arr = (ctypes.c_void_p * len(tensors))(*[_grad_ptr(t, name)[0] for t in tensors])

    @property
    def ptr(self):
        return ctypes.cast(self.arr, ctypes.c_void_p)


def _multi_common(ps, gs):
    if len(ps) == 0:
        return None, None, None, None
    dev = ps[0].device
    g = _TypedPtrList(gs, "g")
    narr = (ctypes.c_int64 * len(ps))(*[p.numel() for p in ps])
    return dev, g.dtype, g.arr, narr


def dt8_sgd_step_multi(ps, gs, m_codes, m_absmax, lr, momentum, weight_decay, step, block_size=2048,
                       stream=None) -> None:
    _check_list_layout("dt8_sgd_step_multi", block_size, ps, gs, m_codes, m_absmax)
    dev, gd, garr, narr = _multi_common(ps, gs)
    if dev is None:
        return
    pl = _TypedPtrList(ps, "p")
    mc = _PtrList(m_codes, torch.uint8, "m_codes")
    ma = _PtrList(m_absmax, torch.float32, "m_absmax")
    with _on_device(dev):
        st = load_library().dt8_sgd_step_multi_ex(
            len(ps), pl.ptr, pl.dtype, ctypes.cast(garr, ctypes.c_void_p), gd, mc.ptr, ma.ptr,
            ctypes.cast(narr, ctypes.c_void_p), lr, momentum, weight_decay, step, block_size,
            _stream_ptr(stream, dev))
    _check(st, "dt8_sgd_step_multi")


def dt8_adam_step_multi(ps, gs, m_codes, m_absmax, r_codes, r_absmax, lr, beta1, beta2, eps,
                        weight_decay, step, block_size=2048, flags=DEFAULT_ADAM_FLAGS, stream=None) -> None:
    _check_list_layout("dt8_adam_step_multi", block_size, ps, gs, m_codes, m_absmax, r_codes, r_absmax)
    dev, gd, garr, narr = _multi_common(ps, gs)
    if dev is None:
        return
    pl = _TypedPtrList(ps, "p")
    mc = _PtrList(m_codes, torch.uint8, "m_codes")
    ma = _PtrList(m_absmax, torch.float32, "m_absmax")
    rc = _PtrList(r_codes, torch.uint8, "r_codes")
    ra = _PtrList(r_absmax, torch.float32, "r_absmax")
    with _on_device(dev):
        st = load_library().dt8_adam_step_multi_ex(
            len(ps), pl.ptr, pl.dtype, ctypes.cast(garr, ctypes.c_void_p), gd, mc.ptr, ma.ptr, rc.ptr, ra.ptr,
            ctypes.cast(narr, ctypes.c_void_p), lr, beta1, beta2, eps, weight_decay, step, block_size,
            flags, _stream_ptr(stream, dev))
    _check(st, "dt8_adam_step_multi")


class PreparedTensorList:
    """Pointer arrays of a tensor list, marshalled once and reused for every step.

    The step functions above rebuild the host pointer arrays on each call, which costs more host
    time than the launch itself for a few hundred tensors.  The tensors of an optimizer are updated
    in place, so their addresses do not change between steps: marshal them once here and call
    ``adam_step`` / ``sgd_step`` per step.  The object keeps the tensors alive.  Gradients must be
    written into the same gradient tensors before each step."""

    def __init__(self, ps, gs, m_codes, m_absmax, r_codes=None, r_absmax=None):
        if len(ps) == 0:
            raise ValueError("empty tensor list")
        self._keep = (list(ps), list(gs), list(m_codes), list(m_absmax),
                      list(r_codes or []), list(r_absmax or []))
        self.device, self.g_dtype, self._g, self._n = _multi_common(ps, gs)
        self.num = len(ps)
        self._p = _TypedPtrList(ps, "p")
        self._mc = _PtrList(m_codes, torch.uint8, "m_codes")
        self._ma = _PtrList(m_absmax, torch.float32, "m_absmax")
        self._rc = _PtrList(r_codes, torch.uint8, "r_codes") if r_codes is not None else None
        self._ra = _PtrList(r_absmax, torch.float32, "r_absmax") if r_absmax is not None else None
        self._layout_checked = set()      # block sizes whose state sizes were verified

    def _check_block_size(self, where: str, block_size: int) -> None:
        """The sizes of the states depend on the block size, which arrives with the step: verify
        them the first time a block size is used (the tensors cannot change size afterwards)."""
        if block_size in self._layout_checked:
            return
        ps, gs, mc, ma, rc, ra = self._keep
        _check_list_layout(where, block_size, ps, gs, mc, ma, rc if self._rc is not None else None,
                           ra if self._ra is not None else None)
        self._layout_checked.add(block_size)

    def sgd_step(self, lr, momentum, weight_decay, step, block_size=2048, stream=None) -> None:
        self._check_block_size("PreparedTensorList.sgd_step", block_size)
        with _on_device(self.device):
            st = load_library().dt8_sgd_step_multi_ex(
                self.num, self._p.ptr, self._p.dtype, ctypes.cast(self._g, ctypes.c_void_p), self.g_dtype,
                self._mc.ptr, self._ma.ptr, ctypes.cast(self._n, ctypes.c_void_p), lr, momentum,
                weight_decay, step, block_size, _stream_ptr(stream, self.device))
        _check(st, "dt8_sgd_step_multi")

    def adam_step(self, lr, beta1, beta2, eps, weight_decay, step, block_size=2048,
                  flags=DEFAULT_ADAM_FLAGS, stream=None) -> None:
        if self._rc is None or self._ra is None:
            raise ValueError("this list was prepared without second-moment states")
        self._check_block_size("PreparedTensorList.adam_step", block_size)
        with _on_device(self.device):
            st = load_library().dt8_adam_step_multi_ex(
                self.num, self._p.ptr, self._p.dtype, ctypes.cast(self._g, ctypes.c_void_p), self.g_dtype,
                self._mc.ptr, self._ma.ptr, self._rc.ptr, self._ra.ptr,
                ctypes.cast(self._n, ctypes.c_void_p), lr, beta1, beta2, eps, weight_decay, step,
                block_size, flags, _stream_ptr(stream, self.device))
        _check(st, "dt8_adam_step_multi")


def shard_blocks(num_blocks_total: int, rank: int, world_size: int) -> range:
    """Contiguous range of whole quantization blocks owned by `rank`.

    Every block is quantized on its own (Section IV-B, "Tensor chunking"),
    so a tensor can be split across ranks on block boundaries with no exchange between them.
    The first `num_blocks_total % world_size` ranks own one extra block."""
    if not (0 <= rank < world_size):
        raise ValueError("rank out of range")
    q, r = divmod(num_blocks_total, world_size)
    start = rank * q + min(rank, r)
    return range(start, start + q + (1 if rank < r else 0))

"""dt8 oracle -- TEST INFRASTRUCTURE, NOT THE PRODUCT.

numpy-facing wrapper around ``dt8_oracle.c``, the plain CPU statement of the 8-bit
optimizer step of Section IV of the paper (dynamic-tree data type, Eq. quant1-quant3,
Eq. sgd, Eq. adam).  Only tests, the smoke check and the benchmark's cpu-baseline leg
may import this package; the CUDA library and its Python binding never do, and this
package imports nothing from them.

Parity unpinned: the code-book VALUES (against the cited data type) and the 100-step
quantized trajectory; everything else is pinned by the ``-m "not gpu"`` tests.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "dt8_oracle.c")
_OUT_DIR = os.path.join(_HERE, "_build")
_SO = os.path.join(_OUT_DIR, "libdt8_oracle.so")

FLAG_BIAS_CORRECTION = 1
FLAG_DECOUPLED_WD = 2
DEFAULT_ADAM_FLAGS = FLAG_BIAS_CORRECTION | FLAG_DECOUPLED_WD
F32, BF16 = 0, 1

_lock = threading.Lock()
_lib = None


def _compile(src: str, out: str) -> None:
    tmp = out + ".%d.tmp" % os.getpid()
    cmd = ["gcc", "-O2", "-std=c11", "-ffp-contract=off", "-fno-fast-math", "-fopenmp",
           "-shared", "-fPIC", "-o", tmp, src, "-lm"]
    subprocess.run(cmd, check=True)
    os.replace(tmp, out)


def build_source(src: str, name: str, variant_env: str, force: bool = False) -> str:
    """Compile one C file of the checker with gcc (no contraction, no fast-math) and return the
    .so path.

    The mutation tests set `variant_env` to a deliberately broken copy of the C file to show that
    the pins notice it; that copy is built next to itself (in the test's temporary directory) and
    never replaces the real library."""
    variant = os.environ.get(variant_env)
    if variant:
        out = os.path.splitext(variant)[0] + ".%d.so" % os.getpid()
        _compile(variant, out)
        return out
    os.makedirs(_OUT_DIR, exist_ok=True)
    out = os.path.join(_OUT_DIR, name)
    stale = (not os.path.exists(out)) or os.path.getmtime(out) < os.path.getmtime(src)
    if force or stale:
        _compile(src, out)
    return out


def build(force: bool = False) -> str:
    """Build every C file of the checker; returns the path of the optimizer checker's library."""
    from . import rev
    rev.build(force)
    return build_source(_SRC, "libdt8_oracle.so", "DT8_ORACLE_SOURCE", force)


def _load():
    global _lib
    with _lock:
        if _lib is None:
            lib = ctypes.CDLL(build())
            c = ctypes
            fp, u8p, vp = c.POINTER(c.c_float), c.POINTER(c.c_uint8), c.c_void_p
            lib.dt8o_set_threads.argtypes = [c.c_int]
            lib.dt8o_get_threads.restype = c.c_int
            lib.dt8o_codebook.argtypes = [c.c_int, fp]
            lib.dt8o_nearest_many.argtypes = [fp, fp, c.c_int64, c.c_int, u8p]
            lib.dt8o_quantize_blockwise.argtypes = [fp, c.c_int64, c.c_int, c.c_int, c.c_int, u8p, fp]
            lib.dt8o_dequantize_blockwise.argtypes = [u8p, fp, c.c_int64, c.c_int, c.c_int, fp]
            lib.dt8o_sgd_update_fp32.argtypes = [fp, fp, fp, c.c_int64, c.c_float, c.c_float, c.c_float]
            lib.dt8o_adam_update_fp32.argtypes = [fp, fp, fp, fp, c.c_int64, c.c_float, c.c_float,
                                                  c.c_float, c.c_float, c.c_float, c.c_int64, c.c_uint32]
            lib.dt8o_sgd_step.argtypes = [fp, vp, c.c_int, u8p, fp, c.c_int64, c.c_float, c.c_float,
                                          c.c_float, c.c_int64, c.c_int]
            lib.dt8o_adam_step.argtypes = [fp, vp, c.c_int, u8p, fp, u8p, fp, c.c_int64, c.c_float,
                                           c.c_float, c.c_float, c.c_float, c.c_float, c.c_int64,
                                           c.c_int, c.c_uint32]
            lib.dt8o_sgd_step_ex.argtypes = [vp, c.c_int, vp, c.c_int, u8p, fp, c.c_int64, c.c_float,
                                             c.c_float, c.c_float, c.c_int64, c.c_int]
            lib.dt8o_adam_step_ex.argtypes = [vp, c.c_int, vp, c.c_int, u8p, fp, u8p, fp, c.c_int64,
                                              c.c_float, c.c_float, c.c_float, c.c_float, c.c_float,
                                              c.c_int64, c.c_int, c.c_uint32]
            lib.dt8o_bf16_round_many.argtypes = [fp, c.c_int64, vp]
            _lib = lib
    return _lib


def _f32(a, name):
    if not (isinstance(a, np.ndarray) and a.dtype == np.float32 and a.flags.c_contiguous):
        raise TypeError(f"{name}: need a C-contiguous float32 ndarray")
    return a.ctypes.data_as(ctypes.POINTER(ctypes.c_float))


def _u8(a, name):
    if not (isinstance(a, np.ndarray) and a.dtype == np.uint8 and a.flags.c_contiguous):
        raise TypeError(f"{name}: need a C-contiguous uint8 ndarray")
    return a.ctypes.data_as(ctypes.POINTER(ctypes.c_uint8))


def _grad(g):
    """fp32 ndarray, or bf16 bit patterns as a uint16 ndarray."""
    if not (isinstance(g, np.ndarray) and g.flags.c_contiguous):
        raise TypeError("g: need a C-contiguous ndarray")
    if g.dtype == np.float32:
        return g.ctypes.data_as(ctypes.c_void_p), F32
    if g.dtype == np.uint16:
        return g.ctypes.data_as(ctypes.c_void_p), BF16
    raise TypeError("g: float32, or uint16 holding bfloat16 bit patterns")


def set_threads(t: int) -> None:
    _load().dt8o_set_threads(int(t))


def get_threads() -> int:
    return int(_load().dt8o_get_threads())


def num_blocks(n: int, block_size: int) -> int:
    if block_size < 1:
        raise ValueError("block_size must be positive")
    return (n + block_size - 1) // block_size


def codebook(is_signed: bool) -> np.ndarray:
    """The 256 ascending values of the data type (Section IV-B, Fig. dynamic_tree)."""
    out = np.empty(256, np.float32)
    rc = _load().dt8o_codebook(int(bool(is_signed)), _f32(out, "out"))
    assert rc == 0
    return out


def nearest(Q: np.ndarray, v: np.ndarray, method: str = "bsearch") -> np.ndarray:
    """Eq. quant2 for already-normalised values: 'scan' = exhaustive argmin, 'bsearch'."""
    v = np.ascontiguousarray(v, np.float32).ravel()
    out = np.empty(v.size, np.uint8)
    _load().dt8o_nearest_many(_f32(np.ascontiguousarray(Q, np.float32), "Q"), _f32(v, "v"), v.size,
                              1 if method == "scan" else 0, _u8(out, "out"))
    return out


def quantize_blockwise(x: np.ndarray, block_size: int, is_signed: bool, method: str = "bsearch"):
    """Eq. quant1 + quant2 per block -> (codes uint8[n], absmax float32[ceil(n/B)])."""
    x = np.ascontiguousarray(x, np.float32).ravel()
    codes = np.empty(x.size, np.uint8)
    absmax = np.empty(num_blocks(x.size, block_size), np.float32)
    rc = _load().dt8o_quantize_blockwise(_f32(x, "x"), x.size, block_size, int(bool(is_signed)),
                                         1 if method == "scan" else 0, _u8(codes, "codes"),
                                         _f32(absmax, "absmax"))
    if rc:
        raise ValueError("oracle quantize: bad arguments")
    return codes, absmax


def dequantize_blockwise(codes: np.ndarray, absmax: np.ndarray, block_size: int, is_signed: bool):
    """Eq. quant3 per block."""
    out = np.empty(codes.size, np.float32)
    assert absmax.size == num_blocks(codes.size, block_size)
    rc = _load().dt8o_dequantize_blockwise(_u8(codes, "codes"), _f32(absmax, "absmax"), codes.size,
                                           block_size, int(bool(is_signed)), _f32(out, "out"))
    if rc:
        raise ValueError("oracle dequantize: bad arguments")
    return out


def sgd_update_fp32(w, g, m, lr, momentum, weight_decay):
    """Eq. sgd on exact fp32 state, in place on w and m."""
    _load().dt8o_sgd_update_fp32(_f32(w, "w"), _f32(g, "g"), _f32(m, "m"), w.size, lr, momentum,
                                 weight_decay)


def adam_update_fp32(w, g, m, r, lr, beta1, beta2, eps, weight_decay, step,
                     flags=DEFAULT_ADAM_FLAGS):
    """Eq. adam on exact fp32 state, in place on w, m and r."""
    _load().dt8o_adam_update_fp32(_f32(w, "w"), _f32(g, "g"), _f32(m, "m"), _f32(r, "r"), w.size,
                                  lr, beta1, beta2, eps, weight_decay, step, flags)


def bf16_round(x) -> np.ndarray:
    """binary32 -> bfloat16 bit patterns (uint16), round to nearest even, element by element."""
    x = np.ascontiguousarray(x, np.float32).ravel()
    out = np.empty(x.size, np.uint16)
    _load().dt8o_bf16_round_many(_f32(x, "x"), x.size, out.ctypes.data_as(ctypes.c_void_p))
    return out


def _param(w):
    """fp32 ndarray, or bf16 bit patterns as a uint16 ndarray (the variant without a 32-bit copy)."""
    if not (isinstance(w, np.ndarray) and w.flags.c_contiguous):
        raise TypeError("w: need a C-contiguous ndarray")
    if w.dtype == np.float32:
        return w.ctypes.data_as(ctypes.c_void_p), F32
    if w.dtype == np.uint16:
        return w.ctypes.data_as(ctypes.c_void_p), BF16
    raise TypeError("w: float32, or uint16 holding bfloat16 bit patterns")


def sgd_step(w, g, m_codes, m_absmax, lr, momentum, weight_decay, step, block_size):
    """One 8-bit SGD step, in place on w (fp32, or bf16 bit patterns), m_codes, m_absmax."""
    gp, gd = _grad(g)
    wp, wd_ = _param(w)
    assert g.size == w.size == m_codes.size and m_absmax.size == num_blocks(w.size, block_size)
    rc = _load().dt8o_sgd_step_ex(wp, wd_, gp, gd, _u8(m_codes, "m_codes"),
                                  _f32(m_absmax, "m_absmax"), w.size, lr, momentum, weight_decay,
                                  step, block_size)
    if rc:
        raise ValueError("oracle sgd_step: bad arguments")


def adam_step(w, g, m_codes, m_absmax, r_codes, r_absmax, lr, beta1, beta2, eps, weight_decay,
              step, block_size, flags=DEFAULT_ADAM_FLAGS):
    """One 8-bit Adam/AdamW step, in place on w (fp32, or bf16 bit patterns) and both states."""
    gp, gd = _grad(g)
    wp, wd_ = _param(w)
    nb = num_blocks(w.size, block_size)
    assert g.size == w.size == m_codes.size == r_codes.size
    assert m_absmax.size == nb and r_absmax.size == nb
    rc = _load().dt8o_adam_step_ex(wp, wd_, gp, gd, _u8(m_codes, "m_codes"),
                                   _f32(m_absmax, "m_absmax"), _u8(r_codes, "r_codes"),
                                   _f32(r_absmax, "r_absmax"), w.size, lr, beta1, beta2, eps,
                                   weight_decay, step, block_size, flags)
    if rc:
        raise ValueError("oracle adam_step: bad arguments")


def sgd_step_multi(ws, gs, m_codes, m_absmax, lr, momentum, weight_decay, step, block_size):
    """Tensor list: each tensor stepped on its own; blocks never span tensors."""
    for t in range(len(ws)):
        sgd_step(ws[t], gs[t], m_codes[t], m_absmax[t], lr, momentum, weight_decay, step, block_size)


def adam_step_multi(ws, gs, m_codes, m_absmax, r_codes, r_absmax, lr, beta1, beta2, eps,
                    weight_decay, step, block_size, flags=DEFAULT_ADAM_FLAGS):
    for t in range(len(ws)):
        adam_step(ws[t], gs[t], m_codes[t], m_absmax[t], r_codes[t], r_absmax[t], lr, beta1, beta2,
                  eps, weight_decay, step, block_size, flags)

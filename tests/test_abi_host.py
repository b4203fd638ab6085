"""CPU-side checks of the CUDA library: it loads, exports what include/dt8.h declares, rejects bad
arguments before touching a device, and its host-built tables agree with the CPU checker.
No compute call reaches a GPU here."""
import ctypes
import os
import re

import numpy as np
import pytest

import oracle
import paper_2412_01195_b200 as dt8
from paper_2412_01195_b200 import build as dt8_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    dt8_build.build_library()
    return dt8.load_library()


def declared_symbols():
    import glob
    names = set()
    for path in glob.glob(os.path.join(ROOT, "include", "*.h")):
        text = re.sub(r"/\*.*?\*/", "", open(path).read(), flags=re.S)
        names |= set(re.findall(r"\b(dt8_[a-z0-9_]+)\s*\(", text))
    return sorted(names)


def test_library_exports_every_declared_symbol(lib):
    names = declared_symbols()
    assert {"dt8_codebook", "dt8_quantize_blockwise", "dt8_dequantize_blockwise", "dt8_sgd_step",
            "dt8_adam_step", "dt8_sgd_step_multi", "dt8_adam_step_multi"} <= set(names)
    for name in names:
        assert hasattr(lib, name), name
    from paper_2412_01195_b200 import rev
    assert set(names) == set(dt8.EXPORTS) | set(rev.REV_EXPORTS)
    assert set(rev.REV_EXPORTS) == {n for n in names if n.startswith("dt8_rev_")}


def test_status_strings(lib):
    for code in range(5):
        assert lib.dt8_status_string(code).decode().startswith("DT8_")
    assert b"unknown" in lib.dt8_status_string(99)


@pytest.mark.parametrize("signed", [True, False])
def test_codebook_is_bit_identical_to_the_checker(signed):
    a, b = dt8.dt8_codebook(signed), oracle.codebook(signed)
    assert np.array_equal(a.view(np.uint32), b.view(np.uint32))


def test_state_bytes_and_the_papers_saving(paper_facts):
    """1 byte per element + 4 bytes per block; the paper's "75 %" on its own kind of tensor list."""
    from paper_2412_01195_b200 import synth
    assert dt8.dt8_state_bytes(0) == 0
    assert dt8.dt8_state_bytes(1) == 5 and dt8.dt8_state_bytes(2048) == 2052
    assert dt8.dt8_state_bytes(2049) == 2049 + 8 and dt8.dt8_state_bytes(256, 256) == 260
    with pytest.raises(ValueError):
        dt8.dt8_state_bytes(10, 1000)
    flat_full, flat_small = dt8.optimizer_state_bytes([1 << 28], 2)
    assert flat_full == paper_facts["adam_state_bytes_fp32"] * (1 << 28)
    assert abs(100 * (1 - flat_small / flat_full) - 74.95) < 0.01
    sizes = [synth.numel(s) for _, s, _ in synth.resnet_speaker_manifest()]
    for states in (1, 2):                                  # SGD momentum, Adam
        full, small = dt8.optimizer_state_bytes(sizes, states)
        assert full == 4 * states * sum(sizes)
        saving = 100 * (1 - small / full)
        # small batch-norm vectors pay a whole absmax each, so a real list saves a little less
        assert paper_facts["memory_saving_percent"] - 0.2 < saving < paper_facts["memory_saving_percent"]


def test_codebook_null(lib):
    assert lib.dt8_codebook(1, None) == dt8.DT8_ERR_INVALID_ARG


def ulp_neighbourhood(x32, radius):
    bits = x32.astype(np.float32).view(np.int32).astype(np.int64)
    return np.concatenate([(bits + d).astype(np.int32).view(np.float32) for d in range(-radius, radius + 1)])


@pytest.mark.parametrize("signed", [True, False])
def test_table_encoder_equals_checker_on_critical_inputs(signed):
    Q = oracle.codebook(signed)
    Q64 = Q.astype(np.float64)
    mids = ((Q64[:-1] + Q64[1:]) / 2).astype(np.float32)
    rng = np.random.default_rng(70)
    pools = [Q, ulp_neighbourhood(Q, 8), ulp_neighbourhood(mids, 64), -ulp_neighbourhood(mids, 64),
             rng.uniform(-1, 1, 1_000_000).astype(np.float32),
             (10.0 ** rng.uniform(-12, 0, 500_000) * rng.choice([-1, 1], 500_000)).astype(np.float32),
             np.array([0.0, -0.0, 1.0, -1.0, 1e-38, -1e-38, 1e-45, 2.0, -2.0, 1e30, -1e30], np.float32)]
    for v in pools:
        v = v[np.isfinite(v)]
        assert np.array_equal(dt8.dt8_selfcheck_encode_host(signed, v), oracle.nearest(Q, v))
    # bucket edges of the table: all values whose low 15/16 bits are 0, 1 or all-ones
    expo = np.arange(90, 128, dtype=np.uint32)[:, None, None] << 23
    mant_hi = (np.arange(256, dtype=np.uint32) << 15)[None, :, None]
    low = np.array([0, 1, 2, 0x7FFE, 0x7FFF], np.uint32)[None, None, :]
    edge = (expo | mant_hi | low).ravel().view(np.float32)
    edge = np.concatenate([edge, -edge])
    assert np.array_equal(dt8.dt8_selfcheck_encode_host(signed, edge), oracle.nearest(Q, edge))


@pytest.mark.parametrize("signed", [True, False])
def test_table_encoder_strided_sweep_of_all_floats(signed):
    """Every 61st binary32 bit pattern with |v| <= 1, both signs (about 35 million values)."""
    Q = oracle.codebook(signed)
    bits = np.arange(0, 0x3F800001, 61, dtype=np.uint32)
    for sign in (0, 0x80000000):
        v = (bits | np.uint32(sign)).view(np.float32)
        assert np.array_equal(dt8.dt8_selfcheck_encode_host(signed, v), oracle.nearest(Q, v))


def test_shared_memory_layout_check_accepts_this_build_and_refuses_tables_that_do_not_fit(lib):
    """The kernels address their tables at fixed shared-memory offsets; the host check that
    guards this must pass for the tables of the build and fail for doctored extents."""
    sf, sn, uf, un = ctypes.c_uint32(), ctypes.c_int(), ctypes.c_uint32(), ctypes.c_int()
    assert lib.dt8_selfcheck_table_extents(ctypes.byref(sf), ctypes.byref(sn), ctypes.byref(uf),
                                           ctypes.byref(un)) == dt8.DT8_OK
    fits = lambda a, b, c, d: lib.dt8_selfcheck_layout_fits(a, b, c, d)
    assert fits(sf.value, sn.value, uf.value, un.value) == 1
    assert fits(sf.value, sn.value + 4096, uf.value, un.value) == 0      # signed table runs into the decode tables
    assert fits(sf.value, sn.value, uf.value, un.value + 4096) == 0      # unsigned table runs into the signed one
    assert fits(sf.value, sn.value, uf.value - 8192, un.value) == 0      # unsigned table starts below the scratch
    assert fits(sf.value - 4096, sn.value, uf.value, un.value) == 0      # signed table overlaps the unsigned one
    assert fits(0, 1, 0, 1) == 0 and fits(sf.value, 0, uf.value, un.value) == 0
    assert lib.dt8_selfcheck_table_extents(None, None, None, None) == dt8.DT8_ERR_INVALID_ARG


def test_non_finite_inputs_stay_inside_the_tables():
    v = np.array([np.nan, -np.nan, np.inf, -np.inf, 3e38, -3e38], np.float32)
    for signed in (True, False):
        dt8.dt8_selfcheck_encode_host(signed, v)      # must not crash; values unspecified


def test_argument_checks_return_before_any_device_work(lib):
    """These all fail validation on the host, so they are safe without a GPU."""
    f = lambda x: ctypes.c_float(x)
    buf = (ctypes.c_uint8 * 4096)()
    base = ctypes.addressof(buf)
    base += (-base) % 16
    ok, odd = ctypes.c_void_p(base), ctypes.c_void_p(base + 2)
    E = dt8
    # bad block size / sizes / null pointers / alignment for quantize and dequantize
    assert lib.dt8_quantize_blockwise(ok, 16, 1000, 1, ok, ok, None) == E.DT8_ERR_UNSUPPORTED
    assert lib.dt8_quantize_blockwise(ok, -1, 2048, 1, ok, ok, None) == E.DT8_ERR_INVALID_ARG
    assert lib.dt8_quantize_blockwise(None, 16, 2048, 1, ok, ok, None) == E.DT8_ERR_INVALID_ARG
    assert lib.dt8_quantize_blockwise(odd, 16, 2048, 1, ok, ok, None) == E.DT8_ERR_ALIGNMENT
    assert lib.dt8_quantize_blockwise(ok, 0, 2048, 1, None, None, None) == E.DT8_OK
    assert lib.dt8_dequantize_blockwise(ok, ok, 16, 300, 0, ok, None) == E.DT8_ERR_UNSUPPORTED
    assert lib.dt8_dequantize_blockwise(ok, None, 16, 256, 0, ok, None) == E.DT8_ERR_INVALID_ARG
    assert lib.dt8_dequantize_blockwise(ok, ok, 16, 256, 0, odd, None) == E.DT8_ERR_ALIGNMENT
    assert lib.dt8_dequantize_blockwise(None, None, 0, 256, 0, None, None) == E.DT8_OK
    # sgd
    sgd = lambda p, g, gd, mc, ma, n, step, B: lib.dt8_sgd_step(p, g, gd, mc, ma, n, f(.1), f(.9), f(0), step, B, None)
    assert sgd(ok, ok, 7, ok, ok, 16, 1, 2048) == E.DT8_ERR_INVALID_ARG
    assert sgd(ok, ok, 0, ok, ok, 16, 0, 2048) == E.DT8_ERR_INVALID_ARG
    assert sgd(ok, ok, 0, ok, ok, -5, 1, 2048) == E.DT8_ERR_INVALID_ARG
    assert sgd(ok, ok, 0, ok, ok, 16, 1, 100) == E.DT8_ERR_UNSUPPORTED
    assert sgd(None, ok, 0, ok, ok, 16, 1, 2048) == E.DT8_ERR_INVALID_ARG
    assert sgd(odd, ok, 0, ok, ok, 16, 1, 2048) == E.DT8_ERR_ALIGNMENT
    assert sgd(ok, ok, 0, odd, ok, 16, 1, 2048) == E.DT8_ERR_ALIGNMENT
    assert sgd(None, None, 0, None, None, 0, 1, 2048) == E.DT8_OK
    # adam
    adam = lambda p, g, gd, mc, ma, rc, ra, n, step, B, fl: lib.dt8_adam_step(
        p, g, gd, mc, ma, rc, ra, n, f(1e-3), f(.9), f(.999), f(1e-8), f(0), step, B, fl, None)
    assert adam(ok, ok, 0, ok, ok, ok, ok, 16, 1, 2048, 8) == E.DT8_ERR_INVALID_ARG
    assert adam(ok, ok, 0, ok, ok, ok, ok, 16, 0, 2048, 3) == E.DT8_ERR_INVALID_ARG
    assert adam(ok, ok, 2, ok, ok, ok, ok, 16, 1, 2048, 3) == E.DT8_ERR_INVALID_ARG
    assert adam(ok, ok, 0, ok, ok, None, ok, 16, 1, 2048, 3) == E.DT8_ERR_INVALID_ARG
    assert adam(ok, ok, 0, ok, ok, ok, odd, 16, 1, 2048, 3) == E.DT8_ERR_ALIGNMENT
    assert adam(ok, ok, 0, ok, ok, ok, ok, 16, 1, 4000, 3) == E.DT8_ERR_UNSUPPORTED
    assert adam(None, None, 0, None, None, None, None, 0, 1, 2048, 3) == E.DT8_OK
    # bf16 gradients need only 8-byte alignment
    half = ctypes.c_void_p(base + 8)
    assert adam(ok, half, 0, ok, ok, ok, ok, 16, 1, 2048, 3) == E.DT8_ERR_ALIGNMENT
    # pointer lists
    arr = (ctypes.c_void_p * 2)(base, base)
    bad = (ctypes.c_void_p * 2)(base, base + 2)
    ns = (ctypes.c_int64 * 2)(16, 16)
    neg = (ctypes.c_int64 * 2)(16, -1)
    ap, bp = ctypes.cast(arr, ctypes.c_void_p), ctypes.cast(bad, ctypes.c_void_p)
    nsp, negp = ctypes.cast(ns, ctypes.c_void_p), ctypes.cast(neg, ctypes.c_void_p)
    sgdm = lambda num, p, n, B=2048, step=1: lib.dt8_sgd_step_multi(num, p, ap, 0, ap, ap, n, f(.1), f(.9), f(0), step, B, None)
    assert sgdm(-1, ap, nsp) == E.DT8_ERR_INVALID_ARG
    assert sgdm(0, None, None) == E.DT8_OK
    assert sgdm(2, None, nsp) == E.DT8_ERR_INVALID_ARG
    assert sgdm(2, bp, nsp) == E.DT8_ERR_ALIGNMENT
    assert sgdm(2, ap, negp) == E.DT8_ERR_INVALID_ARG
    assert sgdm(2, ap, nsp, B=77) == E.DT8_ERR_UNSUPPORTED
    assert sgdm(2, ap, nsp, step=0) == E.DT8_ERR_INVALID_ARG
    adamm = lambda num, p, rc, n, fl=3: lib.dt8_adam_step_multi(
        num, p, ap, 0, ap, ap, rc, ap, n, f(1e-3), f(.9), f(.999), f(1e-8), f(0), 1, 2048, fl, None)
    assert adamm(2, ap, None, nsp) == E.DT8_ERR_INVALID_ARG
    assert adamm(2, ap, bp, nsp) == E.DT8_ERR_ALIGNMENT
    assert adamm(2, ap, ap, nsp, fl=4) == E.DT8_ERR_INVALID_ARG
    assert adamm(0, None, None, None) == E.DT8_OK


def test_hyper_parameters_are_validated_before_any_device_work(lib):
    """Non-finite values, decay rates outside [0, 1), negative eps / momentum: argument errors."""
    f = ctypes.c_float
    buf = (ctypes.c_uint8 * 4096)()
    base = ctypes.addressof(buf)
    ok = ctypes.c_void_p(base + (-base) % 16)
    E = dt8
    adam = lambda lr=1e-3, b1=.9, b2=.999, eps=1e-8, wd=0.: lib.dt8_adam_step(
        ok, ok, 0, ok, ok, ok, ok, 16, f(lr), f(b1), f(b2), f(eps), f(wd), 1, 2048, 3, None)
    for kw in (dict(lr=float("nan")), dict(lr=float("inf")), dict(b1=1.0), dict(b2=1.0), dict(b1=-0.1),
               dict(b2=1.5), dict(eps=-1e-8), dict(eps=float("nan")), dict(wd=float("inf"))):
        assert adam(**kw) == E.DT8_ERR_INVALID_ARG, kw
    sgd = lambda lr=.1, mom=.9, wd=0.: lib.dt8_sgd_step(ok, ok, 0, ok, ok, 16, f(lr), f(mom), f(wd), 1, 2048, None)
    for kw in (dict(lr=float("nan")), dict(mom=float("inf")), dict(mom=-0.5), dict(wd=float("nan"))):
        assert sgd(**kw) == E.DT8_ERR_INVALID_ARG, kw
    arr = (ctypes.c_void_p * 1)(ok.value)
    ns = (ctypes.c_int64 * 1)(16)
    ap, nsp = ctypes.cast(arr, ctypes.c_void_p), ctypes.cast(ns, ctypes.c_void_p)
    assert lib.dt8_adam_step_multi(1, ap, ap, 0, ap, ap, ap, ap, nsp, f(1e-3), f(1.0), f(.999), f(1e-8),
                                   f(0), 1, 2048, 3, None) == E.DT8_ERR_INVALID_ARG
    assert lib.dt8_sgd_step_multi(1, ap, ap, 0, ap, ap, nsp, f(float("nan")), f(.9), f(0), 1, 2048,
                                  None) == E.DT8_ERR_INVALID_ARG
    # the pointer-list forms accept as many blocks per tensor as the single-tensor forms do
    big = (ctypes.c_int64 * 1)((0x7FFF0000 + 1) * 256)
    assert lib.dt8_sgd_step_multi(1, ap, ap, 0, ap, ap, ctypes.cast(big, ctypes.c_void_p), f(.1), f(.9),
                                  f(0), 1, 256, None) == E.DT8_ERR_UNSUPPORTED
    assert lib.dt8_sgd_step(ok, ok, 0, ok, ok, (0x7FFF0000 + 1) * 256, f(.1), f(.9), f(0), 1, 256,
                            None) == E.DT8_ERR_UNSUPPORTED


def test_reversible_kernel_argument_checks_return_before_any_device_work(lib):
    from paper_2412_01195_b200 import rev
    rev._lib()
    buf = (ctypes.c_uint8 * 4096)()
    base = ctypes.addressof(buf)
    ok, odd = ctypes.c_void_p(base + (-base) % 16), ctypes.c_void_p(base + (-base) % 16 + 2)
    E = dt8
    for fn in (lib.dt8_rev_coupling_forward, lib.dt8_rev_coupling_inverse):
        assert fn(ok, ok, ok, -1, 8, 0, None) == E.DT8_ERR_INVALID_ARG
        assert fn(ok, ok, ok, 2, -8, 0, None) == E.DT8_ERR_INVALID_ARG
        assert fn(ok, ok, ok, 2, 8, 2, None) == E.DT8_ERR_INVALID_ARG
        assert fn(None, ok, ok, 2, 8, 0, None) == E.DT8_ERR_INVALID_ARG
        assert fn(odd, ok, ok, 2, 8, 0, None) == E.DT8_ERR_ALIGNMENT
        assert fn(None, None, None, 0, 8, 0, None) == E.DT8_OK
    s2d, d2s = lib.dt8_rev_space_to_depth, lib.dt8_rev_depth_to_space
    assert s2d(ok, 1, 1, 3, 4, ok, None) == E.DT8_ERR_INVALID_ARG          # odd F
    assert s2d(ok, 1, 1, 4, 5, ok, None) == E.DT8_ERR_INVALID_ARG          # odd T
    assert s2d(ok, -1, 1, 4, 4, ok, None) == E.DT8_ERR_INVALID_ARG
    assert s2d(None, 1, 1, 4, 4, ok, None) == E.DT8_ERR_INVALID_ARG
    assert s2d(odd, 1, 1, 4, 4, ok, None) == E.DT8_ERR_ALIGNMENT
    assert s2d(ok, 1 << 20, 1 << 10, 4, 4, ok, None) == E.DT8_ERR_UNSUPPORTED   # 2^34 elements
    assert s2d(None, 0, 4, 4, 4, None, None) == E.DT8_OK
    assert d2s(ok, 1, 1, -2, 2, ok, None) == E.DT8_ERR_INVALID_ARG
    assert d2s(None, 1, 4, 0, 2, None, None) == E.DT8_OK


class _NoLaunch:
    """Stands where the loaded library would be: any attempt to call into it fails the test."""

    def __getattr__(self, name):
        raise AssertionError(f"the binding reached the library ({name}) with inconsistent sizes")


def test_binding_refuses_inconsistent_sizes_before_the_call(monkeypatch):
    """A state built for one block size stepped with another, a gradient of another length, a
    state list of another length: the binding raises ValueError and never reaches the library
    (the C ABI takes n and block_size on trust and would write past the absmax array)."""
    import torch
    monkeypatch.setattr(dt8, "_lib", _NoLaunch())
    n, B = 8 * 2048, 2048
    p, g = torch.zeros(n), torch.zeros(n)
    codes = torch.zeros(n, dtype=torch.uint8)
    am = torch.zeros(n // B)
    hp = (1e-3, 0.9, 0.999, 1e-8, 0.0, 1)
    with pytest.raises(ValueError, match="block maxima"):
        dt8.dt8_adam_step(p, g, codes, am, codes, am, *hp, 256)           # state built for B = 2048
    with pytest.raises(ValueError, match="g holds"):
        dt8.dt8_adam_step(p, g[:-1], codes, am, codes, am, *hp, B)
    with pytest.raises(ValueError, match="r_codes holds"):
        dt8.dt8_adam_step(p, g, codes, am, codes[:5], am, *hp, B)
    with pytest.raises(ValueError, match="block_size"):
        dt8.dt8_adam_step(p, g, codes, am, codes, am, *hp, 1000)
    with pytest.raises(ValueError, match="block maxima"):
        dt8.dt8_sgd_step(p, g, codes, am[:-1], 0.1, 0.9, 0.0, 1, B)
    with pytest.raises(ValueError, match="block maxima"):
        dt8.dt8_quantize_blockwise(p, 256, True, codes, am)
    with pytest.raises(ValueError, match="out holds"):
        dt8.dt8_dequantize_blockwise(codes, am, B, True, torch.zeros(n - 1))
    with pytest.raises(ValueError, match="lists 1 tensors"):
        dt8.dt8_adam_step_multi([p, p], [g, g], [codes, codes], [am, am], [codes], [am, am], *hp, B)
    with pytest.raises(ValueError, match=r"m_absmax\[1\]"):
        dt8.dt8_sgd_step_multi([p, p], [g, g], [codes, codes], [am, am[:3]], 0.1, 0.9, 0.0, 1, B)
    with pytest.raises(ValueError, match="is on"):
        dt8._check_layout("x", n, B, torch.device("cuda", 0), {"g": g}, {})
    # consistent sizes pass the layout check and stop at the next one (these are host tensors)
    with pytest.raises(TypeError, match="CUDA tensor"):
        dt8.dt8_adam_step(p, g, codes, am, codes, am, *hp, B)


def test_binding_fails_loudly_without_the_library(monkeypatch, tmp_path):
    monkeypatch.setattr(dt8, "_lib", None)
    monkeypatch.setattr(dt8, "_LIB_PATH", str(tmp_path / "nope.so"))
    with pytest.raises(RuntimeError, match="no fallback"):
        dt8.dt8_codebook(True)


def test_shard_blocks_partitions_exactly():
    for nb in (0, 1, 7, 131072, 3437):
        for world in (1, 2, 3, 8):
            seen = []
            for r in range(world):
                seen += list(dt8.shard_blocks(nb, r, world))
            assert seen == list(range(nb))
            sizes = [len(dt8.shard_blocks(nb, r, world)) for r in range(world)]
            assert max(sizes) - min(sizes) <= 1
    with pytest.raises(ValueError):
        dt8.shard_blocks(10, 2, 2)

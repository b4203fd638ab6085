"""Host-side checks of bench.py: the launch path for --gpus N (run here with two gloo ranks and
no GPU work), the byte models, and the rule for the reported DRAM traffic."""
import json
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import bench  # noqa: E402


def _run(args, env=None):
    e = dict(os.environ)
    for k in ("RANK", "WORLD_SIZE", "LOCAL_RANK", "MASTER_ADDR", "MASTER_PORT"):
        e.pop(k, None)
    e.update(env or {})
    return subprocess.run([sys.executable, os.path.join(ROOT, "bench.py")] + args, cwd=ROOT, env=e,
                          capture_output=True, text=True, timeout=600)


def test_gpus_2_without_a_launcher_starts_two_ranks():
    """Started the way the driver starts the N = 1 run but with --gpus 2: the script launches two
    ranks of itself, they meet over the process group, and the line says n_gpus = 2."""
    p = _run(["--gpus", "2", "--plumbing-check"])
    assert p.returncode == 0, p.stderr[-2000:]
    lines = [ln for ln in p.stdout.splitlines() if ln.startswith("{")]
    assert len(lines) == 1, p.stdout
    out = json.loads(lines[0])
    assert out["n_gpus"] == 2 and out["slowest"] == 2.0


def test_a_line_never_claims_fewer_gpus_than_asked():
    """One rank under a launcher's environment but --gpus 2: refused, nothing printed."""
    p = _run(["--gpus", "2", "--plumbing-check"],
             env={"RANK": "0", "WORLD_SIZE": "1", "LOCAL_RANK": "0", "MASTER_ADDR": "127.0.0.1", "MASTER_PORT": "29999"})
    assert p.returncode != 0
    assert "rank(s) are running" in p.stderr
    assert not [ln for ln in p.stdout.splitlines() if ln.startswith("{")]


def test_byte_models():
    n, B = 1 << 20, 2048
    assert bench.adam_bytes(n, B) == 16 * n + 16 * (n // B)
    assert bench.adam_bytes(n, B, g_bytes=2) == 14 * n + 16 * (n // B)
    assert bench.adam_bytes(n, B, g_bytes=2, p_bytes=2) == 10 * n + 16 * (n // B)
    assert bench.sgd_bytes(n, B) == 14 * n + 8 * (n // B)
    assert bench.sgd_bytes(n + 1, B) == 14 * (n + 1) + 8 * (n // B + 1)


def test_traffic_is_null_once_the_kernel_sources_changed(monkeypatch):
    monkeypatch.setitem(bench.NCU_CAPTURE, "source_hash", "0" * 16)
    traffic, note = bench.reported_traffic(1 << 28, 2048)
    assert traffic is None and "changed" in note
    monkeypatch.setitem(bench.NCU_CAPTURE, "source_hash", bench.kernel_source_hash())
    traffic, _ = bench.reported_traffic(1 << 28, 2048)
    cap = bench.NCU_CAPTURE["dram_read"] + bench.NCU_CAPTURE["dram_write"]
    assert traffic == cap + bench.adam_bytes(1 << 28, 2048) - bench.adam_bytes(1 << 26, 2048)
    # at the captured size the figure is the capture itself
    assert bench.reported_traffic(1 << 26, 2048)[0] == cap


def test_every_default_sub_case_exists():
    pytest.importorskip("torch")
    assert set(bench.DEFAULT_SUBS) <= set(bench.sub_cases())

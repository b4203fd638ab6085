"""Do the pins notice a mistake?  Each case plants one plausible mistake in a COPY of the CPU
checker's C source (a dropped term, a wrong sign or index, a reciprocal instead of a division, the
wrong table ...), builds it, and runs the checker's pin tests against it in a child process: the
pins must fail.  Nothing here touches the CUDA path, and the real checker is never replaced."""
import os
import subprocess
import sys
from concurrent.futures import ThreadPoolExecutor

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
SRC = os.path.join(ROOT, "oracle", "dt8_oracle.c")
REV_SRC = os.path.join(ROOT, "oracle", "rev_oracle.c")
PIN_FILES = ["tests/test_oracle_codebook.py", "tests/test_oracle_quant.py", "tests/test_oracle_updates.py",
             "tests/test_oracle_bf16_params.py"]
REV_PIN_FILES = ["tests/test_oracle_rev.py"]

# (name, text in the source, replacement)
MUTANTS = [
    ("fraction off by one", "9 * ((int64_t)k + 1)", "9 * ((int64_t)k)"),
    ("negative half not negated", "out[127 - p] = -v;", "out[127 - p] = v;"),
    ("decade scale one power short", "for (int i = 0; i <= E; ++i) den *= 10;", "for (int i = 0; i < E; ++i) den *= 10;"),
    ("scan ties to the higher index", "if (d < bestd) { bestd = d; best = j; }", "if (d <= bestd) { bestd = d; best = j; }"),
    ("bisection ties to the higher index", "j = (dhi < dlo) ? hi : lo;", "j = (dhi <= dlo) ? hi : lo;"),
    ("reciprocal instead of division", "float v = (N > 0.0f) ? x[i] / N : 0.0f;", "float v = (N > 0.0f) ? x[i] * (1.0f / N) : 0.0f;"),
    ("maximum of signed values", "float a = fabsf(x[i]);", "float a = x[i];"),
    ("dequantize without the block maximum", "out[i] = Q[codes[i]] * N;", "out[i] = Q[codes[i]];"),
    ("momentum sign", "float mi = beta * m[i] + gi;", "float mi = beta * m[i] - gi;"),
    ("sgd ascent", "w[i] = w[i] - lr * mi;", "w[i] = w[i] + lr * mi;"),
    ("sgd decay dropped", "if (wd != 0.0f) gi = gi + wd * w[i];", "if (wd != 0.0f) gi = gi;"),
    ("second moment of g instead of g^2", "float ri = beta2 * r[i] + omb2 * (gi * gi);", "float ri = beta2 * r[i] + omb2 * gi;"),
    ("first moment without (1 - beta1)", "float mi = beta1 * m[i] + omb1 * gi;", "float mi = beta1 * m[i] + gi;"),
    ("eps inside the root", "float upd = mhat / (sqrtf(rhat) + eps);", "float upd = mhat / sqrtf(rhat + eps);"),
    ("decoupled decay dropped", "if (flags & DT8O_FLAG_DECOUPLED_WD) wi = wi * decay;", "if (flags & DT8O_FLAG_DECOUPLED_WD) wi = wi;"),
    ("bias correction with the wrong beta", "*bc2 = (float)(1.0 - pow((double)beta2, (double)step));", "*bc2 = (float)(1.0 - pow((double)beta1, (double)step));"),
    ("second moment on the signed table", "quantize_block(Qu, r, cnt, 0, r_codes + s, r_absmax + b);", "quantize_block(Qs, r, cnt, 0, r_codes + s, r_absmax + b);"),
    ("second moment decoded with the signed table", "dequantize_block(Qu, r_codes + s, r_absmax[b], cnt, r);", "dequantize_block(Qs, r_codes + s, r_absmax[b], cnt, r);"),
    ("bf16 widened into the low half", "uint32_t u = (uint32_t)h << 16;", "uint32_t u = (uint32_t)h;"),
    ("bf16 store truncates", "if (dropped > 0x8000u || (dropped == 0x8000u && (kept & 1u))) kept += 1;", "(void)dropped;"),
    ("bf16 store rounds half up", "(dropped == 0x8000u && (kept & 1u))", "(dropped == 0x8000u)"),
    ("parameter halved when read in the Adam step", "for (int i = 0; i < cnt; ++i) wb[i] = param_at(w, p_dtype, s + i);\n    dequantize_block(Qs, m_codes + s, m_absmax[b], cnt, m);\n    dequantize_block(Qu,", "for (int i = 0; i < cnt; ++i) wb[i] = 0.5f * param_at(w, p_dtype, s + i);\n    dequantize_block(Qs, m_codes + s, m_absmax[b], cnt, m);\n    dequantize_block(Qu,"),
]

# mistakes planted in the checker of the reversible-network kernels
REV_MUTANTS = [
    ("row and column offsets swapped", "const int64_t co = c * r * r + df * r + dt;", "const int64_t co = c * r * r + dt * r + df;"),
    ("block-major channel order", "const int64_t co = c * r * r + df * r + dt;", "const int64_t co = (df * r + dt) * C + c;"),
    ("inverse rearrangement reads the wrong offset", "const int64_t c = co / (r * r), df = (co % (r * r)) / r, dt = co % r;", "const int64_t c = co / (r * r), dt = (co % (r * r)) / r, df = co % r;"),
    ("inverse coupling adds", "o[i] = sign > 0 ? a[i] + b[i] : a[i] - b[i];", "o[i] = a[i] + b[i];"),
    ("coupling takes the other half", "const float *a = in + (2 * n + which) * half;", "const float *a = in + (2 * n + 1 - which) * half;"),
    ("branch output indexed like the full tensor", "const float *b = t + n * half;", "const float *b = t + 2 * n * half;"),
]


def _run_pins(tmp_dir, idx, name, old, new, src=SRC, env_name="DT8_ORACLE_SOURCE", pin_files=PIN_FILES):
    text = open(src).read()
    assert text.count(old) == 1, f"mutant {name!r}: the text to replace occurs {text.count(old)} times"
    path = os.path.join(tmp_dir, f"mutant_{idx}.c")
    with open(path, "w") as fh:
        fh.write(text.replace(old, new))
    env = dict(os.environ, OMP_NUM_THREADS="2")
    env[env_name] = path
    cmd = [sys.executable, "-m", "pytest", *pin_files, "-x", "-q", "-p", "no:cacheprovider",
           "-k", "not trajectory_stays_near"]
    proc = subprocess.run(cmd, cwd=ROOT, env=env, capture_output=True, text=True, timeout=900)
    return name, proc.returncode, proc.stdout[-400:]


def test_every_planted_mistake_is_noticed(tmp_path):
    with ThreadPoolExecutor(max_workers=6) as pool:
        results = list(pool.map(lambda a: _run_pins(str(tmp_path), *a),
                                [(i, *m) for i, m in enumerate(MUTANTS)]))
    survived = [name for name, rc, _ in results if rc == 0]
    broken = [(name, out) for name, rc, out in results if rc not in (0, 1)]
    assert not broken, f"pin run did not complete: {broken}"
    assert not survived, f"no pin noticed: {survived}"


def test_the_unmodified_source_passes_as_a_variant(tmp_path):
    """Control: the same child-process run on an unmodified copy passes, so a failure above is due
    to the planted mistake and not to the harness."""
    name, rc, out = _run_pins(str(tmp_path), 99, "control", "float a = fabsf(x[i]);", "float a = fabsf(x[i]);")
    assert rc == 0, out


def test_every_planted_mistake_in_the_reversible_kernels_checker_is_noticed(tmp_path):
    args = dict(src=REV_SRC, env_name="REV_ORACLE_SOURCE", pin_files=REV_PIN_FILES)
    with ThreadPoolExecutor(max_workers=6) as pool:
        results = list(pool.map(lambda a: _run_pins(str(tmp_path), *a, **args),
                                [(i, *m) for i, m in enumerate(REV_MUTANTS)]))
    survived = [name for name, rc, _ in results if rc == 0]
    broken = [(name, out) for name, rc, out in results if rc not in (0, 1)]
    assert not broken, f"pin run did not complete: {broken}"
    assert not survived, f"no pin noticed: {survived}"
    name, rc, out = _run_pins(str(tmp_path), 99, "control", "int which, int sign) {", "int which, int sign) {", **args)
    assert rc == 0, out

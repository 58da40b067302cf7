"""Do the pins catch plausible mistakes?  Each case plants one mistake in a COPY of the oracle's C source (a wrong
sign, a swapped operand, a dropped rounding rule, a wrong index, ...), builds it on the CPU and runs the oracle's pin
tests against that copy: at least one pin must fail.  A mutant that survives means a pin is missing."""
import os
import shutil
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
PINS = ["tests/test_oracle_haar.py", "tests/test_oracle_select_quant.py", "tests/test_oracle_layer.py",
        "tests/test_oracle_options.py", "tests/test_oracle_wavelets.py"]

# (file, text as it stands, text with the mistake)
MUTANTS = [
    ("wcc_oracle_impl.h", "const REAL s0 = a + b, d0 = a - b, s1 = c + d, d1 = c - d;", "const REAL s0 = a + b, d0 = b - a, s1 = c + d, d1 = c - d;"),
    ("wcc_oracle_impl.h", "dst[(size_t)i * W + j + w]       = (d0 + d1) * half;", "dst[(size_t)i * W + j + w]       = (s0 - s1) * half;"),
    ("wcc_oracle_impl.h", "dst[(size_t)(i + h) * W + j + w] = (d0 - d1) * half;", "dst[(size_t)(i + h) * W + j + w] = (d0 + d1) * half;"),
    ("wcc_oracle_impl.h", "dst[(size_t)(2 * i) * W + 2 * j + 1]     = (t0 - u0) * half;", "dst[(size_t)(2 * i) * W + 2 * j + 1]     = (t0 + u0) * half;"),
    ("wcc_oracle_impl.h", "const REAL half = (REAL)0.5;\n    for (int i = 0; i < h; ++i) {\n        for (int j = 0; j < w; ++j) {\n            const REAL a", "const REAL half = (REAL)0.25;\n    for (int i = 0; i < h; ++i) {\n        for (int j = 0; j < w; ++j) {\n            const REAL a"),
    ("wcc_oracle_impl.h", "acc = FMA(v, v, acc);", "acc = acc + v * v;"),
    ("wcc_oracle_impl.h", "for (int c = 0; c < C; ++c) {\n                const REAL v = coef", "for (int c = C - 1; c >= 0; --c) {\n                const REAL v = coef"),
    ("wcc_oracle_impl.h", "return (a->p > b->p) - (a->p < b->p);", "return (a->p < b->p) - (a->p > b->p);"),
    ("wcc_oracle_impl.h", "if (a->v > b->v) return -1;\n    if (a->v < b->v) return 1;", "if (a->v > b->v) return 1;\n    if (a->v < b->v) return -1;"),
    ("wcc_oracle_impl.h", "if (tau) tau[n] = a[k - 1].v;", "if (tau) tau[n] = a[k].v;"),
    ("wcc_oracle.c", "float r = nearbyintf(x[i] * inv);", "float r = roundf(x[i] * inv);"),
    ("wcc_oracle.c", "return amax / qmax;", "return amax / (qmax + 1.0f);"),
    ("wcc_oracle.c", "const float qmax = (float)((1 << (bits - 1)) - 1);\n    const float amax = alpha;", "const float qmax = (float)(1 << (bits - 1));\n    const float amax = alpha;"),
    ("wcc_oracle.c", "if (r < -qmax) r = -qmax;", "if (r < -qmax - 1.0f) r = -qmax - 1.0f;"),
    ("wcc_oracle.c", "Yc[(size_t)r * Cout + o] = (float)acc * (scale_a * scale_w[o]);", "Yc[(size_t)r * Cout + o] = (float)acc * (scale_a * scale_w[0]);"),
    ("wcc_oracle.c", "Xc[((size_t)n * k + j) * Cin + c] = coef[((size_t)n * Cin + c) * P + idx[(size_t)n * k + j]];", "Xc[((size_t)n * k + j) * Cin + c] = coef[((size_t)n * Cin + c) * P + idx[(size_t)j]];"),
    ("wcc_oracle.c", "acc += (int32_t)Wq[(size_t)o * Cin + c] * (int32_t)Xq[(size_t)r * Cin + c];", "acc += (int32_t)Wq[(size_t)c * Cout + o] * (int32_t)Xq[(size_t)r * Cin + c];"),
    ("wcc_oracle.c", "y[i] = y[i] + residual[i];", "y[i] = y[i] - residual[i];"),
    ("wcc_oracle.c", "y[i] = (y[i] > 0.0f) ? y[i] : 0.0f;", "y[i] = (y[i] < 0.0f) ? y[i] : 0.0f;"),
    ("wcc_oracle.c", "if (residual)\n        for (size_t i = 0; i < (size_t)N * Cout * P; ++i) y[i] = y[i] + residual[i];\n    if (relu)\n        for (size_t i = 0; i < (size_t)N * Cout * P; ++i) y[i] = (y[i] > 0.0f) ? y[i] : 0.0f;",
     "if (relu)\n        for (size_t i = 0; i < (size_t)N * Cout * P; ++i) y[i] = (y[i] > 0.0f) ? y[i] : 0.0f;\n    if (residual)\n        for (size_t i = 0; i < (size_t)N * Cout * P; ++i) y[i] = y[i] + residual[i];"),
    ("wcc_oracle.c", "orc_quantize_alpha(Xc, (long)(nk * Cin), bits, alpha, Xq)", "orc_quantize_alpha(Xc, (long)(nk * Cin), bits, 2.0f * alpha, Xq)"),
    ("wcc_oracle.c", "orc_quantize_weights(Wt, Cout, Cin, wbits, Wq, scale_w);", "orc_quantize_weights(Wt, Cout, Cin, bits, Wq, scale_w);"),
    ("wcc_oracle.c", "const int rr = r + i - 1, cc = c + j - 1;", "const int rr = r - i + 1, cc = c + j - 1;"),
    ("wcc_oracle.c", "u += 0x7FFFu + lsb;", "u += 0x8000u;"),
    ("wcc_oracle_impl.h", "if (mr & 1) continue;", "if (!(mr & 1)) continue;"),
    ("wcc_oracle_impl.h", "const int cc = ((2 * j + tc - c0) % wc + wc) % wc;", "const int cc = ((2 * j + tc) % wc + wc) % wc;"),
    ("wcc_oracle_impl.h", "out[(b * T + tr) * T + tc] = ((b >> 1) ? hi[tr] : lo[tr]) * ((b & 1) ? hi[tc] : lo[tc]);", "out[(b * T + tr) * T + tc] = ((b & 1) ? hi[tr] : lo[tr]) * ((b >> 1) ? hi[tc] : lo[tc]);"),
]


@pytest.mark.parametrize("case", range(len(MUTANTS)), ids=lambda i: "mutant%02d" % i)
def test_a_planted_mistake_is_caught(case, tmp_path):
    fname, good, bad = MUTANTS[case]
    src_dir = os.path.join(ROOT, "oracle")
    for f in ("wcc_oracle.c", "wcc_oracle_impl.h"):
        shutil.copy(os.path.join(src_dir, f), tmp_path / f)
    text = (tmp_path / fname).read_text()
    assert text.count(good) == 1, "the oracle's source changed: update this mutant"
    (tmp_path / fname).write_text(text.replace(good, bad))
    lib = str(tmp_path / "liboracle_mutant.so")
    subprocess.check_call(["gcc", "-std=c11", "-O1", "-ffp-contract=off", "-fno-fast-math", "-fopenmp", "-shared", "-fPIC",
                           "-o", lib, str(tmp_path / "wcc_oracle.c"), "-lm"])
    env = dict(os.environ, WCC_ORACLE_LIB=lib, OMP_NUM_THREADS="2")
    r = subprocess.run([sys.executable, "-m", "pytest", "-x", "-q", "-m", "not gpu", "-p", "no:cacheprovider"] + PINS,
                       cwd=ROOT, env=env, stdout=subprocess.PIPE, stderr=subprocess.STDOUT, text=True)
    assert r.returncode != 0, "this mistake went unnoticed by every pin:\n%s\n->\n%s" % (good, bad)

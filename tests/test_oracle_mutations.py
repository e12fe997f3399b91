"""The pins have teeth: single-token mutations of the oracle each fail at least one pin.

Every mutation below is one plausible mistake (a tie direction, an off-by-one scale, the wrong
one of several equal maxima, a dropped term, a floating-point shortcut).  A mutated copy of
mxp_oracle.c is compiled to a temporary library and the pin files are run against it in a
child process; the child must FAIL.  The unmutated source, run the same way, must pass.
No GPU."""
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
SRC = os.path.join(ROOT, "oracle", "mxp_oracle.c")
T = "tests/"

# (name, text in the source, replacement, pin files that must notice)
MUTATIONS = [
    ("nbm_ties_to_odd_code", "if (d < best_d || (d == best_d && (c & 1) == 0)) {\n            best = c;\n            best_d = d;\n        }\n    }\n    /* 7.0 is midway",
     "if (d < best_d || (d == best_d && (c & 1) == 1)) {\n            best = c;\n            best_d = d;\n        }\n    }\n    /* 7.0 is midway", [T + "test_oracle_format.py"]),
    ("bm_ties_away_from_even", "if (frac > 0.5 || (frac == 0.5 && (m & 1)))\n        m += 1;\n    if (m > 7)",
     "if (frac >= 0.5)\n        m += 1;\n    if (m > 7)", [T + "test_oracle_format.py"]),
    ("scale_off_by_one", "int se = floor_log2(amax) - EMAX;", "int se = floor_log2(amax) - EMAX + 1;", [T + "test_oracle_format.py"]),
    ("last_of_equal_maxima", "        if (a > amax) {\n            amax = a;\n            bm = i;\n        }\n    }\n    memset(nib, 0, (size_t)k / 2);",
     "        if (a >= amax) {\n            amax = a;\n            bm = i;\n        }\n    }\n    memset(nib, 0, (size_t)k / 2);", [T + "test_oracle_format.py"]),
    ("bm_decode_step", "out = ldexp(ldexp(1.0 + (double)code / 8.0, EMAX), sb - 127);",
     "out = ldexp(ldexp(1.0 + (double)code / 4.0, EMAX), sb - 127);", [T + "test_oracle_format.py"]),
    ("flush_boundary", "if (amax == 0.0 || floor_log2(amax) <= -127 + EMAX) {", "if (amax == 0.0 || floor_log2(amax) < -127 + EMAX) {",
     [T + "test_oracle_format.py"]),
    ("gemm_transposed_operand", "acc += A[m * lda + kk] * B[n * ldb + kk];", "acc += A[m * lda + kk] * B[kk * ldb + n];",
     [T + "test_oracle_gemm.py"]),
    ("mxpp_offset_dropped", "int e = max2 - EMAX + 1;", "int e = max2 - EMAX;", [T + "test_oracle_mxpp.py"]),
    ("wide_bm_clamp_dropped", None, None, [T + "test_oracle_wide.py"]),   # filled in below
    ("nvfp4_reciprocal_in_binary32", "double v = fabs(x[i]) / d;", "double v = (double)((float)fabs(x[i]) * (1.0f / (float)d));",
     [T + "test_oracle_nvfp4.py"]),
    ("nvfp4_scale_maps_bm_to_4", "amax / (6.0 * ts)", "amax / (4.0 * ts)", [T + "test_oracle_nvfp4.py"]),
    ("nvfp4_fallback_threshold", "int extend = plus && sb > 2;\n    for (int i = 0; i < 16; ++i) {\n        double v", "int extend = plus && sb > 1;\n    for (int i = 0; i < 16; ++i) {\n        double v",
     [T + "test_oracle_nvfp4.py"]),
]


def _source():
    with open(SRC) as f:
        return f.read()


def _wide_clamp(src):
    # the clamp of a wide BM that rounds into the next binade: "if (m > limit) m = limit"
    i = src.index("static int bm_code_wide(int fmt, double v)")
    j = src.index("return m;", i)
    body = src[i:j]
    k = body.rindex("if (m >")
    return body[k:], "/* clamp dropped */\n    "


def _run_pins(lib, files):
    env = dict(os.environ, MXP_ORACLE_LIB=lib, PYTHONPATH=ROOT)
    return subprocess.run([sys.executable, "-m", "pytest", "-x", "-q", "-m", "not gpu", "-p", "no:cacheprovider"] + files,
                          cwd=ROOT, env=env, stdout=subprocess.PIPE, stderr=subprocess.STDOUT, text=True)


def _compile(text, path_c, path_so):
    with open(path_c, "w") as f:
        f.write(text)
    subprocess.check_call(["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-fopenmp", "-fno-fast-math",
                           "-ffp-contract=off", path_c, "-o", path_so, "-lm"])


def test_unmutated_source_passes_the_same_way(tmp_path):
    so = str(tmp_path / "clean.so")
    _compile(_source(), str(tmp_path / "clean.c"), so)
    r = _run_pins(so, [T + "test_oracle_gemm.py", T + "test_oracle_mxpp.py"])
    assert r.returncode == 0, r.stdout[-2000:]


@pytest.mark.parametrize("name,old,new,pins", MUTATIONS, ids=[m[0] for m in MUTATIONS])
def test_mutation_is_caught(name, old, new, pins, tmp_path):
    src = _source()
    if old is None:
        old, new = _wide_clamp(src)
    assert src.count(old) == 1, "mutation site of %s not found exactly once" % name
    so = str(tmp_path / (name + ".so"))
    _compile(src.replace(old, new), str(tmp_path / (name + ".c")), so)
    r = _run_pins(so, pins)
    assert r.returncode == 1, "pins did not notice %s:\n%s" % (name, r.stdout[-1500:])
    assert " failed" in r.stdout

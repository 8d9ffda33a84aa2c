"""The pins have teeth: a planted mistake in the oracle's source makes them fail.

Each case rewrites one expression of ``oracle/rapid_oracle.c`` (on the CPU, in
a temporary copy), builds it, and runs the oracle's pin tests against that
build in a child process; the run must fail.
"""
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
SRC = os.path.join(ROOT, "oracle", "rapid_oracle.c")

MUTATIONS = {
    "mask_off_by_one": ("const int64_t lim = L - R + i;", "const int64_t lim = L - R + i + 1 < L ? L - R + i + 1 : L - 1;"),
    "scale_dropped": ("s[j] = scale * dot;", "s[j] = dot;"),
    "wrong_kv_head": ("const int kvh = h / G;", "const int kvh = h % Hkv;"),
    "value_row_shifted": ("const uint16_t* vrow = vbase + j * kv_stride_l;",
                          "const uint16_t* vrow = vbase + (j > 0 ? j - 1 : 0) * kv_stride_l;"),
    "shift_sign": ("zhat[j] = zd[j] + eta * T * (q[j] - p[j]);", "zhat[j] = zd[j] + eta * T * (p[j] - q[j]);"),
    "shift_without_T": ("zhat[j] = zd[j] + eta * T * (q[j] - p[j]);", "zhat[j] = zd[j] + eta * (q[j] - p[j]);"),
    "tail_keeps_q": ("if (phat[j] < thresh) phat[j] = p[j];", "if (phat[j] < thresh) phat[j] = q[j];"),
    "tail_inverted": ("if (phat[j] < thresh) phat[j] = p[j];", "if (phat[j] > thresh) phat[j] = p[j];"),
    "residual_min": ("r = a > b ? a : b;", "r = a > b ? b : a;"),
    "residual_unclamped": ("w[j] = r > 0.0 ? r : 0.0;", "w[j] = r;"),
    "residual_drops_phat_term": ("const double a = p[j] - phat[j];", "const double a = p[j] - q[j];"),
    "cdf_boundary": ("if (c > target) return j;", "if (c >= target) return j;"),
    "bonus_row_wrong": ("const float* z = target_logits + ((int64_t)b * R + gamma) * V;",
                        "const float* z = target_logits + ((int64_t)b * R + (gamma > 0 ? gamma - 1 : 0)) * V;"),
    "temperature_forgotten": ("out[j] = exp(x[j] / T - m);", "out[j] = exp(x[j] - m * T);"),
    "ratio_uses_p": ("const double ratio = q[x] > 0.0 ? phat[x] / q[x] : INFINITY;",
                     "const double ratio = q[x] > 0.0 ? p[x] / q[x] : INFINITY;"),
    "sampling_uniform_reused": ("const double u = (double)uniforms[(int64_t)b * R + gamma];",
                                "const double u = (double)uniforms[(int64_t)b * R + (n < gamma ? n : gamma)];"),
    "keeps_going_after_reject": ("rejected = 1;\n", "rejected = 0; n = 0;\n"),
    "e4m3_bias_off_by_one": ("else v = ldexp(1.0 + (double)m / 8.0, e - 7);", "else v = ldexp(1.0 + (double)m / 8.0, e - 8);"),
    "e4m3_subnormal_as_normal": ("if (e == 0) v = ldexp((double)m, -9);", "if (e == 0) v = ldexp(1.0 + (double)m / 8.0, -7);"),
    "fp8_value_scale_taken_from_keys": ("const double vs = (double)v_scale[(int64_t)b * Hkv + head8];",
                                        "const double vs = (double)k_scale[(int64_t)b * Hkv + head8];"),
    "fp8_scale_of_the_wrong_head": ("const double ks = (double)k_scale[(int64_t)b * Hkv + head8];",
                                    "const double ks = (double)k_scale[(int64_t)b * Hkv];"),
    "window_one_key_too_narrow": ("if (!(j < sink || j > own - window)) continue;\n            const double e",
                                  "if (!(j < sink || j > own - window + 1)) continue;\n            const double e"),
    "window_anchored_at_last_row": ("const int64_t own = L - R + i; /* the row's own key */",
                                    "const int64_t own = L - 1; /* the row's own key */"),
    "sinks_dropped_from_values": ("if (!(j < sink || j > own - window)) continue;\n            const double e",
                                  "if (!(j > own - window)) continue;\n            const double e"),
}


@pytest.mark.parametrize("name", sorted(MUTATIONS))
def test_planted_mistake_is_caught(name, tmp_path):
    old, new = MUTATIONS[name]
    src = open(SRC).read()
    assert src.count(old) == 1, f"mutation anchor for {name} not unique"
    mutated = tmp_path / "mut.c"
    mutated.write_text(src.replace(old, new))
    lib = tmp_path / "libmut.so"
    subprocess.run(["gcc", "-O1", "-fopenmp", "-shared", "-fPIC", "-o", str(lib), str(mutated), "-lm"], check=True)
    env = dict(os.environ, RAPID_ORACLE_LIB=str(lib))
    r = subprocess.run([sys.executable, "-m", "pytest", "-x", "-q", "-p", "no:cacheprovider",
                        os.path.join(ROOT, "tests", "test_oracle_attention.py"),
                        os.path.join(ROOT, "tests", "test_oracle_accept.py")],
                       env=env, cwd=ROOT, capture_output=True, text=True)
    assert r.returncode != 0, f"pins did not notice the planted mistake '{name}'"

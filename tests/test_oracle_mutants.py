"""The pins must notice plausible mistakes in the oracle.

Each mutant is a one-token edit of the oracle's C source (a dropped term, a wrong sign or
index, a transposed operand, a misplaced scale).  It is compiled into a temporary library
and the pin suite is run against it in a child process; the suite has to fail.  Mistakes
are planted on the CPU only.
"""
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
SRC = os.path.join(ROOT, "oracle", "agent_attention_oracle.c")

MUTANTS = [
    ("scale_also_applied_to_bias",
     "double v = dot * scale;\n            if (bias) v += bias[(size_t)i * cols + j];",
     "double v = dot;\n            if (bias) v += bias[(size_t)i * cols + j];\n            v *= scale;"),
    ("bias_transposed", "bias[(size_t)i * cols + j]", "bias[(size_t)j * rows + i]"),
    ("bias_dropped", "if (bias) v += bias", "if (0) v += bias"),
    ("softmax_not_normalised", "s[j] /= den;", "s[j] /= 1.0;"),
    ("pool_sum_not_mean", "a[c] /= cnt;", "a[c] /= 1.0;"),
    ("pool_window_floor_end", "int x1 = ((ax + 1) * W + pw - 1) / pw;", "int x1 = ((ax + 1) * W) / pw;"),
    ("pool_agent_order_transposed", "A + (size_t)(ay * pw + ax) * d", "A + (size_t)(ax * ph + ay) * d"),
    ("dwc_filter_flipped", "int yy = y + u - 1;", "int yy = y - u + 1;"),
    ("dwc_taps_transposed", "Wd[(size_t)c * 9 + u * 3 + v]", "Wd[(size_t)c * 9 + v * 3 + u]"),
    ("dwc_wraps_rows", "if (xx < 0 || xx >= W) continue;", "if (yy * W + xx < 0 || yy * W + xx >= H * W) continue;"),
    ("scales_swapped", "n, N, d, d, scale1, va, NULL", "n, N, d, d, scale2, va, NULL"),
    ("bias_head_offset_dropped", "b1 ? b1 + (size_t)head * n * N : NULL", "b1 ? b1 : NULL"),
    ("b2_head_offset_dropped", "b2 ? b2 + (size_t)head * N * n : NULL", "b2 ? b2 : NULL"),
    ("dwc_head_offset_dropped", "wd + (size_t)head * d * 9", "wd"),
    ("broadcast_uses_v_not_va", "aa_oracle_softmax_attention(q, a, va,", "aa_oracle_softmax_attention(q, a, v,"),
    ("bias_block_align_corners", "double sy = ((double)y + 0.5) * (double)h0 / (double)h - 0.5;", "double sy = (double)y * (double)(h0 - 1) / (double)(h > 1 ? h - 1 : 1);"),
    ("bias_row_col_swapped", "if (row) v += row[(size_t)a * h + y];", "if (row) v += row[(size_t)a * h + (x < h ? x : h - 1)];"),
    ("bias_transpose_ignored", "if (transpose) out[(size_t)t * n + a] = v;", "if (0) out[(size_t)t * n + a] = v;"),
    ("eq7_aggregation_halved", "p[2] = 2 * n * N * C;", "p[2] = n * N * C;"),
]


@pytest.mark.parametrize("name,old,new", MUTANTS, ids=[m[0] for m in MUTANTS])
def test_pins_catch_mutant(tmp_path, name, old, new):
    src = open(SRC).read()
    assert src.count(old) == 1, "mutation site must be unique in the oracle source"
    mutated = tmp_path / "mutant.c"
    mutated.write_text(src.replace(old, new))
    lib = tmp_path / "libmutant.so"
    subprocess.check_call(["gcc", "-O1", "-fopenmp", "-shared", "-fPIC", "-o", str(lib),
                           str(mutated), "-lm"])
    env = dict(os.environ, AGENT_ATTENTION_ORACLE_LIB=str(lib))
    r = subprocess.run([sys.executable, "-m", "pytest", "-x", "-q", "-p", "no:cacheprovider",
                        os.path.join(ROOT, "tests", "test_oracle_pins.py")],
                       env=env, cwd=ROOT, stdout=subprocess.PIPE, stderr=subprocess.STDOUT)
    assert r.returncode != 0, f"pins did not notice mutant '{name}'"


# The same for the backward oracle: each mutant must fail the backward pins (finite differences of the
# forward oracle, the adjoint identity, the closed forms).
BACKWARD_PINS = os.path.join(ROOT, "tests", "test_oracle_backward_pins.py")
BACKWARD_MUTANTS = [
    ("bwd_broadcast_softmax_jacobian_without_row_term",
     "p2[(size_t)i * n + r] * (ds[(size_t)i * n + r] - dot)", "p2[(size_t)i * n + r] * (ds[(size_t)i * n + r])"),
    ("bwd_aggregation_softmax_jacobian_without_row_term",
     "p1[(size_t)r * N + j] * (ds[(size_t)r * N + j] - dot)", "p1[(size_t)r * N + j] * (ds[(size_t)r * N + j])"),
    ("bwd_dq_wrong_scale", "gq[(size_t)i * d + c] = scale2 * acc;", "gq[(size_t)i * d + c] = scale1 * acc;"),
    ("bwd_dk_wrong_scale", "gk[(size_t)j * d + c] = scale1 * gk_acc;", "gk[(size_t)j * d + c] = scale2 * gk_acc;"),
    ("bwd_agent_gradient_loses_broadcast_term",
     "da[(size_t)r * d + c] += scale1 * acc;", "da[(size_t)r * d + c] = scale1 * acc;"),
    ("bwd_dv_uses_logit_gradient",
     "gv_acc += p1[(size_t)r * N + j] * dva[(size_t)r * d + c];", "gv_acc += ds[(size_t)r * N + j] * dva[(size_t)r * d + c];"),
    ("bwd_depthwise_not_transposed",
     "const int yy = y + u - 1, xx = x + t - 1;", "const int yy = y - u + 1, xx = x - t + 1;"),
    ("bwd_pooling_sum_not_mean",
     "da[(size_t)(ay * pw + ax) * d + c] * inv;", "da[(size_t)(ay * pw + ax) * d + c] * 1.0;"),
    ("bwd_bias_gradient_not_summed_over_batch",
     "if (dB2) dB2[head * nN + (size_t)i * n + r] += g;", "if (dB2) dB2[head * nN + (size_t)i * n + r] = g;"),
]


@pytest.mark.parametrize("name,old,new", BACKWARD_MUTANTS, ids=[m[0] for m in BACKWARD_MUTANTS])
def test_backward_pins_catch_mutant(tmp_path, name, old, new):
    src = open(SRC).read()
    assert src.count(old) == 1, "mutation site must be unique in the oracle source"
    mutated = tmp_path / "mutant.c"
    mutated.write_text(src.replace(old, new))
    lib = tmp_path / "libmutant.so"
    subprocess.check_call(["gcc", "-O1", "-fopenmp", "-shared", "-fPIC", "-o", str(lib),
                           str(mutated), "-lm"])
    env = dict(os.environ, AGENT_ATTENTION_ORACLE_LIB=str(lib))
    r = subprocess.run([sys.executable, "-m", "pytest", "-x", "-q", "-p", "no:cacheprovider", BACKWARD_PINS],
                       env=env, cwd=ROOT, stdout=subprocess.PIPE, stderr=subprocess.STDOUT)
    assert r.returncode != 0, f"backward pins did not notice mutant '{name}'"

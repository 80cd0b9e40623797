"""The pins must be able to fail: plant one plausible mistake at a time in a temporary copy
of the oracle's C source (dropped term, wrong sign, wrong comparison, wrong index), build it,
and check that at least one pin in test_oracle_pins.py then fails.  The mistakes are planted
in the CPU oracle only; nothing here touches a GPU."""
import os
import subprocess
import sys

import pytest

import oracle

SRC = os.path.join(os.path.dirname(oracle.__file__), "picospec_oracle.c")

# (name, text to find, replacement)
MUTANTS = [
    ("tie_break_reversed", "return (x->v > y->v) - (x->v < y->v);", "return (x->v < y->v) - (x->v > y->v);"),
    ("sort_ascending", "if (x->l > y->l) return -1;\n    if (x->l < y->l) return 1;",
     "if (x->l > y->l) return 1;\n    if (x->l < y->l) return -1;"),
    ("temperature_multiplied", "double x = (double)l[v] / T;", "double x = (double)l[v] * T;"),
    ("top_p_strict", "if (cum >= top_p) {", "if (cum > top_p + 0.05) {"),
    ("top_p_off_by_one", "n = j + 1;\n                break;", "n = j + 2 < k_eff ? j + 2 : k_eff;\n                break;"),
    ("no_renormalise", "prob[j] = (float)((w[keys[j].v] / Z) / s);", "prob[j] = (float)(w[keys[j].v] / Z);"),
    ("residual_sign", "double d = w[v] / Z - qd[v];", "double d = qd[v] - w[v] / Z;"),
    ("residual_no_clamp", "r[v] = d > 0.0 ? d : 0.0;", "r[v] = d > 0.0 ? d : -d;"),
    ("residual_drops_q", "for (int j = 0; j < n; ++j) qd[idx[j]] = (double)prob[j];", ";"),
    ("ratio_inverted", "double ratio = px / qx;", "double ratio = qx / px;"),
    ("accept_without_min", "acc = u < lim;", "acc = u * 0.5 < lim;"),
    ("scan_counts_all_accepts", "else\n                            still = 0;", "else\n                            still = 1;"),
    ("borderline_counts_all", "if (still) {\n                        nborder += border;",
     "nborder += border;\n                    if (still) {"),
    ("sampler_level1_nonstrict", "if (cum > thr1) {", "if (cum >= thr1 * 1.2) {"),
    ("sampler_level2_uses_u1", "double thr2 = u2 * M[cs];", "double thr2 = u1 * M[cs];"),
    ("sampler_chunk_offset", "long v0 = cs * chunk, v1 = v0 + chunk < V ? v0 + chunk : V;\n    long tok",
     "long v0 = 0, v1 = chunk < V ? chunk : V;\n    long tok"),
    ("bonus_uses_residual", "int resid = a < G;", "int resid = a < G + 1 && a > 0 ? 1 : a < G;"),
    ("sample_wrong_row", "long t = pso_sample_row(rows + a * row_stride,", "long t = pso_sample_row(rows + 0 * row_stride,"),
    ("px_wrong_index", "double px = w[x] / Z;", "double px = w[(x + 1) % V] / Z;"),
    ("draw_nonstrict", "if (cum > thr) return idx[j];", "if (cum >= thr * 1.3) return idx[j];"),
    ("topk_renormalised", "prob[t] = (float)(w[keys[t].v] / Z);", "prob[t] = (float)(w[keys[t].v] / Z * 1.5);"),
    ("topk_wrong_row", "const float *l = target_logits + (b * rows_per_seq + j) * row_stride;",
     "const float *l = target_logits + (b * rows_per_seq + 0) * row_stride;"),
    ("edge_residual_sign", "double d = (double)prob[t] - w[idx[t]] / Z;", "double d = w[idx[t]] / Z - (double)prob[t];"),
    ("edge_ignores_q", "double d = (double)prob[t] - w[idx[t]] / Z;", "double d = (double)prob[t];"),
    ("edge_wrong_row", "const float *l = draft_logits + (b * rows_per_seq + j) * row_stride;",
     "const float *l = draft_logits + (b * rows_per_seq + 0) * row_stride;"),
    ("edge_nonstrict", "if (cum > thr) {\n                        pick = t;", "if (cum >= thr * 1.2) {\n                        pick = t;"),
    ("range_restarts_at_zero", "long a = r0;", "long a = 0;"),
    ("range_bonus_before_its_row", "int bonus = ok && !rejected && g < r1;", "int bonus = ok && !rejected;"),
    ("range_ignores_gamma", "long g = gamma ? gamma[b] : G;", "long g = G;"),
    ("range_ignores_state", "if (state_in && state_in[b] == 0) {", "if (0) {"),
    ("range_reads_later_rows", "long hi = g < r1 ? g : r1;", "long hi = g;"),
    ("vanished_residual_threshold_too_high", "if (R > PSO_RESID_ZERO) tok", "if (R > 1e-9) tok"),
    ("vanished_residual_never", "if (R > PSO_RESID_ZERO) tok", "if (R > 0.0) tok"),
    ("edge_no_fallback", "if (!(R > 0.0)) {\n                    R = 0.0;", "if (0) {\n                    R = 0.0;"),
]

PINS = os.path.join(os.path.dirname(os.path.abspath(__file__)), "test_oracle_pins.py")


@pytest.mark.parametrize("name,old,new", MUTANTS, ids=[m[0] for m in MUTANTS])
def test_planted_mistake_is_caught(name, old, new, tmp_path):
    src = open(SRC).read()
    assert src.count(old) >= 1, f"mutant {name}: pattern not found"
    c = tmp_path / "mutant.c"
    so = tmp_path / "mutant.so"
    c.write_text(src.replace(old, new, 1))
    subprocess.run(["gcc", "-O1", "-std=c11", "-fPIC", "-shared", "-fopenmp", "-ffp-contract=off",
                    "-o", str(so), str(c), "-lm"], check=True)
    # a separate process: a planted mistake may also crash, which counts as noticed
    env = dict(os.environ, PICOSPEC_ORACLE_LIB=str(so))
    run = subprocess.run([sys.executable, "-m", "pytest", PINS, "-x", "-q", "-p", "no:cacheprovider"],
                         env=env, capture_output=True, text=True, timeout=600)
    assert run.returncode != 0, f"no pin noticed the planted mistake '{name}'"

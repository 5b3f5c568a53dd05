"""Each pin of the oracle is shown to bite: a deliberately broken copy of oracle/bebop_oracle.c (one plausible
slip per copy: a dropped term, a wrong sign, an off-by-one, p and q exchanged, a wrong row) is built in a
temporary directory and the pin that is meant to catch that slip is run against it in a child process.  The pin
must fail on the broken build; the regular run of tests/test_oracle_pins.py shows it passing on the real one.
`test_restated_formulas_agree` re-types the oracle's own expressions and is never the pin relied on."""
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
SRC = os.path.join(ROOT, "oracle", "bebop_oracle.c")

# (what the slip is, text to find, replacement, the pin that must catch it)
MUTATIONS = [
    ("bonus drawn from the last drafted row instead of the row after it",
     "st |= oracle_softmax(target + (int64_t)L * ld_t, V, tau, p);\n        if (st & ST_FATAL) goto fatal;",
     "st |= oracle_softmax(target + (int64_t)(L > 0 ? L - 1 : 0) * ld_t, V, tau, p);\n        if (st & ST_FATAL) goto fatal;",
     "test_brute_force_measure_is_exactly_p"),
    ("residual taken as max(0, q - p)",
     "double d = p[v] - q[v]; r[v] = d > 0.0 ? d : 0.0;",
     "double d = q[v] - p[v]; r[v] = d > 0.0 ? d : 0.0;",
     "test_brute_force_measure_is_exactly_p"),
    ("inverse CDF returns the token after the crossing",
     "if (C >= t) { y = v; break; }",
     "if (C >= t) { y = v + 1 < V ? v + 1 : v; break; }",
     "test_inverse_cdf_matches_cumsum_searchsorted"),
    ("accept test with p and q exchanged",
     "double lhs = (double)u_acc[k] * qx;",
     "double lhs = (double)u_acc[k] * px; px = qx;",
     "test_brute_force_measure_is_exactly_p"),
    ("accept on equality (u q <= p) instead of strict",
     "if (lhs >= px) {",
     "if (lhs > px) {",
     "test_zero_residual_falls_back_to_target"),
    ("a stray term in the residual-mass form of TV",
     "a += (d > 0.0) ? d : 0.0;",
     "a += (d > 0.0) ? d : 0.0; a += 1e-9;",
     "test_tv_three_forms_agree_and_bounds"),
    ("temperature multiplied instead of divided",
     "double x = (double)z[v] / tau;\n        prob[v]",
     "double x = (double)z[v] * tau;\n        prob[v]",
     "test_softmax_matches_scipy"),
    ("argmax ties go to the highest index",
     "if (z[v] > m) { m = z[v]; arg = v; }",
     "if (z[v] >= m) { m = z[v]; arg = v; }",
     "test_greedy_reduces_to_leading_argmax_match"),
    ("S of Eq. tv_grad sums p instead of q",
     "if (q[v] <= p[v]) S += q[v];",
     "if (q[v] <= p[v]) S += p[v];",
     "test_s_aux_is_the_scalar_of_the_tv_gradient"),
    ("S of Eq. tv_grad summed over the complementary set",
     "if (q[v] <= p[v]) S += q[v];",
     "if (q[v] > p[v]) S += q[v];",
     "test_golden_dyadic_s_aux_and_margins"),
    ("CDF margin relative to the target u Z instead of the chosen token's mass",
     "*margin_tok = (r[y] > 0.0) ? (double)(gap / (long double)r[y]) : 0.0;",
     "*margin_tok = (t > 0.0L) ? (double)(gap / t) : 0.0;",
     "test_golden_dyadic_s_aux_and_margins"),
    ("accept margin relative to p alone",
     "margin_acc[k] = big > 0.0 ? fabs(lhs - px) / big : 0.0;",
     "margin_acc[k] = px > 0.0 ? fabs(lhs - px) / px : 0.0;",
     "test_golden_dyadic_s_aux_and_margins"),
    ("TV no longer clamped to [0, 1] and the clamp's input negated",
     "tv[k] = clamp01(t3[0]);",
     "tv[k] = -t3[0];",
     "test_golden_dyadic_s_aux_and_margins"),
]


def _run_pin(pin, lib):
    env = dict(os.environ, BEBOP_ORACLE_LIB=lib)
    return subprocess.run([sys.executable, "-m", "pytest", os.path.join(ROOT, "tests", "test_oracle_pins.py"), "-x", "-q",
                           "-p", "no:cacheprovider", "-k", pin], cwd=ROOT, env=env, capture_output=True, text=True)


@pytest.mark.parametrize("what,find,replace,pin", MUTATIONS, ids=[m[0] for m in MUTATIONS])
def test_a_plausible_slip_fails_its_pin(tmp_path, what, find, replace, pin):
    assert pin != "test_restated_formulas_agree"
    src = open(SRC).read()
    assert src.count(find) == 1, "the oracle no longer contains the line this mutation edits: " + find
    mutated = tmp_path / "bebop_oracle_mutated.c"
    mutated.write_text(src.replace(find, replace))
    lib = str(tmp_path / "libmutated.so")
    subprocess.run(["gcc", "-O2", "-std=c11", "-fopenmp", "-fPIC", "-shared", "-o", lib, str(mutated), "-lm"], check=True)
    r = _run_pin(pin, lib)
    assert r.returncode == 1 and " failed" in r.stdout, "the pin %s did not notice: %s\n%s" % (pin, what, r.stdout[-800:])

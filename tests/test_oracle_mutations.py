"""The pins must notice a broken checker.

Each case plants one plausible mistake in a copy of ``oracle/pg_oracle.c`` (on
the CPU, never in the CUDA path), points the binding at the copy and runs the
pin tests in a child process: they have to fail.
"""
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
SRC = os.path.join(ROOT, "oracle", "pg_oracle.c")

MUTATIONS = {
    "update_not_antisymmetric": ("Xj[(size_t)r * m + cidx] += d;", "Xj[(size_t)r * m + cidx] -= d;"),
    "weight_dropped": ("double a = w[e] * p[r];", "double a = p[r];"),
    "left_factor_not_normalised": ("p[r] = ok ? p[r] * inv : 0.0;", "p[r] = ok ? p[r] : 0.0;"),
    "right_vector_not_refreshed": ("memcpy(c->Q[t] + (size_t)k * m, q, sizeof(double) * (size_t)m);", ";"),
    "difference_sign_in_transposed_pass": ("Qn[(size_t)k * m + e] = qi[e] - qj[e];",
                                           "Qn[(size_t)k * m + e] = qi[e] + qj[e];"),
    "forward_uses_one_endpoint": ("p[r] = pi[r] - pj[r];", "p[r] = pi[r];"),
    "no_orthogonalisation": ("for (int r = 0; r < n; ++r) p[r] -= a * ph[r];", ";"),
    "transposed_index": ("for (int cidx = 0; cidx < m; ++cidx) y[cidx] += a[cidx] * vr;",
                         "for (int cidx = 0; cidx < m; ++cidx) y[cidx] += a[cidx] * v[(r + 1) % n];"),
    "matching_weight_is_one": ("for (int e = 0; e < E; ++e) w_out[e] = 0.5;",
                                              "for (int e = 0; e < E; ++e) w_out[e] = 1.0;"),
    "ring_skips_wraparound": ("edges_out[2 * n + 1] = (i + 1) % N; ++n; }",
                              "edges_out[2 * n + 1] = (i + 1) % N; if (i + 1 < N) ++n; }"),
    "philox_round_count": ("round < 10; ++round", "round < 9; ++round"),
    # rank > 1: the dependent-column rule
    "dependent_rule_comparison_flipped": ("(k == 0 || nn > 1e-10 * pre);\n        if (k > 0",
                                          "(k == 0 || nn < 1e-10 * pre);\n        if (k > 0"),
    "dependent_rule_threshold_far_lower": ("(k == 0 || nn > 1e-10 * pre);\n        if (k > 0",
                                           "(k == 0 || nn > 1e-20 * pre);\n        if (k > 0"),
    "dependent_rule_threshold_far_higher": ("(k == 0 || nn > 1e-10 * pre);\n        if (k > 0",
                                            "(k == 0 || nn > 1e-5 * pre);\n        if (k > 0"),
    "dependent_rule_not_relative": ("(k == 0 || nn > 1e-10 * pre);\n        if (k > 0",
                                    "(k == 0 || nn > 1e-10);\n        if (k > 0"),
    "dropped_column_loses_its_vector": ("if (!live[u * (size_t)rank + k]) continue;", ";"),
    # Algorithm 2 read literally (half-step mode)
    "half_step_parity_swapped": ("const int odd = (int)(c->iteration % 2);",
                                 "const int odd = (int)(c->iteration % 2 == 0);"),
    "half_step_vector_not_normalised": ("vh[u][a] = (nv > 0.0 && isfinite(nv)) ? v[a] / nv : 0.0;",
                                        "vh[u][a] = v[a];"),
    "half_step_vector_not_moved": ("memcpy(c->Q[t], out[u], sizeof(double) * (size_t)(odd ? n : m));", ";"),
    "half_step_update_not_antisymmetric": ("Xj[(size_t)r * m + cidx] = Xj[(size_t)r * m + cidx] + d;",
                                           "Xj[(size_t)r * m + cidx] = Xj[(size_t)r * m + cidx] - d;"),
    # random-projection compressors
    "random_directions_not_fresh": ("pgo_random_directions(c->seed, c->step, i, j, l, len_in, rank, dirs[u]);",
                                    "pgo_random_directions(c->seed, 0, i, j, l, len_in, rank, dirs[u]);"),
    "random_directions_not_orthogonalised": ("for (int e = 0; e < len; ++e) u[e] -= a * uh[e];", ";"),
    "random_projection_left_uses_forward_product": (
        "else       { matvec_t(Xi, n, m, d, o); matvec_t(Xj, n, m, d, tmp); }",
        "else       { matvec_t(Xi, n, m, d, o); matvec_t(Xi, n, m, d, tmp); }"),
    "half_step_transposed_operand": ("else     { matvec_t(Xi, n, m, vh[u], pi); matvec_t(Xj, n, m, vh[u], pj); }",
                                     "else     { matvec_t(Xi, n, m, vh[u], pi); matvec_t(Xi, n, m, vh[u], pj); }"),
}


@pytest.mark.parametrize("name", sorted(MUTATIONS))
def test_pins_catch(name, tmp_path):
    old, new = MUTATIONS[name]
    text = open(SRC).read()
    assert text.count(old) == 1, "mutation anchor must be unique: %r" % old
    mutated = tmp_path / "pg_oracle_mutated.c"
    mutated.write_text(text.replace(old, new))
    env = dict(os.environ)
    env["PG_ORACLE_SRC"] = str(mutated)
    env["PG_ORACLE_BUILD"] = str(tmp_path / "build")
    env["OMP_NUM_THREADS"] = "2"
    r = subprocess.run([sys.executable, "-m", "pytest", "-x", "-q", "-p", "no:cacheprovider",
                        os.path.join(ROOT, "tests", "test_oracle_pins.py")],
                       cwd=ROOT, env=env, stdout=subprocess.PIPE, stderr=subprocess.STDOUT, timeout=600)
    assert r.returncode != 0, "pins did not notice mutation %s" % name
    assert b"failed" in r.stdout

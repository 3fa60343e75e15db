"""The pins must bite: each plausible mistake, planted in a copy of the oracle's source on the CPU,
has to make at least one pin fail."""
import os
import subprocess
import sys

import pytest

from oracle.build import SOURCE, compile_source

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

# (name, text in bns_oracle.c, replacement)
MUTANTS = [
    ("bessel_variance", "const double Var = sq / s;", "const double Var = sq / (s - 1.0);"),
    ("eps_outside_root", "const double istd = 1.0 / sqrt(Var + eps);\n        mean[j] = E;",
     "const double istd = 1.0 / (sqrt(Var) + eps);\n        mean[j] = E;"),
    ("dropped_variance_term", "v += dl_dE * (1.0 / s) + dl_dVar * (2.0 * (xi - E) / s);", "v += dl_dE * (1.0 / s);"),
    ("mean_term_sign", "v += dl_dE * (1.0 / s) +", "v += -dl_dE * (1.0 / s) +"),
    ("correction_over_m", "v += dl_dE * (1.0 / s) + dl_dVar * (2.0 * (xi - E) / s);",
     "v += dl_dE * (1.0 / ((double)N * H * W)) + dl_dVar * (2.0 * (xi - E) / ((double)N * H * W));"),
    ("correction_everywhere", "if (in_S(sp, C, n, c, h, w))\n                            v +=", "v +="),
    ("sums_over_sampled_set_only",
     "double dl_dxhat = dyi * g;\n                    dl_dE +=",
     "double dl_dxhat = dyi * g;\n                    if (!in_S(sp, C, n, c, h, w)) continue;\n                    dl_dE +="),
    ("patch_axes_swapped", "return h >= oh && h < oh + sp->ph && w >= ow && w < ow + sp->pw;",
     "return h >= ow && h < ow + sp->ph && w >= oh && w < oh + sp->pw;"),
    ("patch_end_off_by_one", "h < oh + sp->ph &&", "h <= oh + sp->ph &&"),
    ("per_map_index_transposed", "e = (size_t)n * C + c;", "e = (size_t)c + (size_t)n;"),
    ("xhat_without_centering", "dl_dgamma += dyi * ((xi - E) * istd);\n                    dl_dbeta += dyi;\n                }\n        if (virt",
     "dl_dgamma += dyi * (xi * istd);\n                    dl_dbeta += dyi;\n                }\n        if (virt"),
    ("virtual_rows_not_in_sums", "if (virt && dyv)", "if (0 && dyv)"),
    # Eq. 4 and Appendix D
    ("mixed_weights_swapped", "const double E = b * E_v + (1.0 - b) * E_s;", "const double E = b * E_s + (1.0 - b) * E_v;"),
    ("mixed_correction_about_mixed_mean", "v += dl_dE_s / s_s + dl_dVar_s * 2.0 * (xi - E_s) / s_s;",
     "v += dl_dE_s / s_s + dl_dVar_s * 2.0 * (xi - E) / s_s;"),
    ("mixed_virtual_share_dropped", "const double dl_dE_v = b * dl_dE, dl_dVar_v = b * dl_dVar;",
     "const double dl_dE_v = dl_dE, dl_dVar_v = dl_dVar;"),
    ("moving_average_alpha_on_old_value", "alpha * X[c] + (1.0 - alpha) * X_ma[c]", "(1.0 - alpha) * X[c] + alpha * X_ma[c]"),
    ("inference_eps_outside_root", "/ sqrt(Var_ma[c] + eps);", "/ (sqrt(Var_ma[c]) + eps);"),
]


@pytest.mark.parametrize("name,old,new", MUTANTS, ids=[m[0] for m in MUTANTS])
def test_planted_mistake_is_caught(tmp_path, name, old, new):
    text = open(SOURCE).read()
    assert text.count(old) >= 1, f"mutation site for {name} not found"
    src = tmp_path / "mutant.c"
    src.write_text(text.replace(old, new, 1))
    lib = tmp_path / "libmutant.so"
    compile_source(str(src), str(lib))
    env = dict(os.environ, BNS_ORACLE_LIBRARY=str(lib))
    run = subprocess.run([sys.executable, "-m", "pytest", "-x", "-q", "-p", "no:cacheprovider",
                          os.path.join(ROOT, "tests", "test_oracle_pins.py"),
                          os.path.join(ROOT, "tests", "test_oracle_next_rows.py")],
                         cwd=ROOT, env=env, capture_output=True, text=True)
    assert run.returncode != 0, f"no pin noticed the planted mistake '{name}'"
    assert "failed" in run.stdout

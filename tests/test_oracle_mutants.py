"""Mutation check of the pins: a plausible mistake planted in a COPY of the oracle (on the CPU)
must make at least one pin fail.  Each mutant is one textual edit of rib_oracle.c."""
import os
import subprocess
import sys
from pathlib import Path

import pytest

ROOT = Path(__file__).resolve().parent.parent
SRC = (ROOT / "oracle" / "rib_oracle.c").read_text()

MUTANTS = {
    "dropped_rank_scale": ("s[j] = content * inv_sqrt_d + bias * inv_sqrt_r;",
                           "s[j] = content * inv_sqrt_d + bias;"),
    "dropped_bias_term": ("s[j] = content * inv_sqrt_d + bias * inv_sqrt_r;",
                          "s[j] = content * inv_sqrt_d;"),
    "transposed_bias": ("bias += pq[(long)i * sh->r + c] * pk[(long)j * sh->r + c];",
                        "bias += pq[(long)j * sh->r + c] * pk[(long)i * sh->r + c];"),
    "shift_sign": ("*Y = (wy * window + y + shift) % H;",
                   "*Y = (wy * window + y - shift + H) % H;"),
    "column_major_tokens": ("int y = i / window, x = i % window;",
                            "int x = i / window, y = i % window;"),
    "full_width_scale": ("const double inv_sqrt_d = 1.0 / sqrt((double)sh->d);",
                         "const double inv_sqrt_d = 1.0 / sqrt((double)sh->d * sh->heads);"),
    "softmax_no_normalise": ("for (int j = 0; j < n; ++j) p[j] /= sum;",
                             "for (int j = 0; j < n; ++j) p[j] /= (sum * 1.0000001);"),
    "dk_missing_scale": ("dkw[(long)j * d + c] += ds * qw[(long)i * d + c] * inv_sqrt_d;",
                         "dkw[(long)j * d + c] += ds * qw[(long)i * d + c];"),
    "dpk_uses_pk": ("gpk[(long)j * r + c] += ds * pqh[(long)i * r + c] * inv_sqrt_r;",
                    "gpk[(long)j * r + c] += ds * pkh[(long)i * r + c] * inv_sqrt_r;"),
    "ds_without_row_term": ("const double ds = p[j] * (dp[j] - Di);",
                            "const double ds = p[j] * dp[j];"),
    "dv_transposed": ("dvw[(long)j * d + c] += p[j] * gw[(long)i * d + c];",
                      "dvw[(long)i * d + c] += p[j] * gw[(long)j * d + c];"),
}


@pytest.mark.parametrize("name", sorted(MUTANTS))
def test_pins_catch_mutant(name, tmp_path):
    old, new = MUTANTS[name]
    assert SRC.count(old) == 1, "mutation target must occur exactly once"
    mutant = tmp_path / "rib_oracle_mutant.c"
    mutant.write_text(SRC.replace(old, new))
    env = dict(os.environ, RIB_ORACLE_SRC=str(mutant))
    run = subprocess.run([sys.executable, "-m", "pytest", str(ROOT / "tests" / "test_oracle_pins.py"),
                          "-x", "-q", "-p", "no:cacheprovider"], cwd=ROOT, env=env,
                         capture_output=True, text=True)
    assert run.returncode == 1, f"pins did not catch mutant {name}:\n{run.stdout[-2000:]}"

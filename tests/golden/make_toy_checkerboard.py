"""Writes toy_checkerboard.txt from the closed form of the paper's Fig. 1(b) toy (no RoPE case).

A 32x32 map tiles two orthogonal 32-d vectors a, b with |a|^2 = |b|^2 = alpha, Q = K, no
positional term.  A query sees n/2 keys of its own kind with logit alpha/sqrt(d) and n/2 of the
other kind with logit 0, hence the values below.  Uses the math module only.
"""
import math
from pathlib import Path

M, d, alpha = 32, 32, 8.0
n = M * M
e = math.exp(alpha / math.sqrt(d))
p_same = e / ((n / 2) * (e + 1.0))
p_diff = 1.0 / ((n / 2) * (e + 1.0))
lines = [
    "# Closed form of the repeated-pattern toy of Fig. 1(b) (checkerboard attention, no RoPE).",
    "# p_same / p_diff = exp(alpha / sqrt(d)); totals are summed over the n/2 keys of each kind.",
    f"M={M}", f"d={d}", f"alpha={alpha!r}",
    f"p_same_total={(n / 2) * p_same!r}", f"p_diff_total={(n / 2) * p_diff!r}",
    f"lse={math.log((n / 2) * (e + 1.0))!r}",
]
Path(__file__).with_name("toy_checkerboard.txt").write_text("\n".join(lines) + "\n")

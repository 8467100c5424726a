"""CPU oracle for the RIB feature generator (Eq. 1, Eq. 2, Eq. 3).  TEST INFRASTRUCTURE ONLY.

Plain numpy in float64, one statement per step of the paper, and the chain rule of those steps for
the backward pass.  Only the tests, the smoke check and the benchmark's CPU leg may import it; the
CUDA library shares no code with it.

Readings where the paper is silent (parity unpinned on these two points: the paper prints no
worked example of the coordinates):
  * normalised coordinates: M points from -1 to 1 inclusive on both axes (a single point sits at 0);
    token i = y * M + x of the window has coordinate (row coordinate, column coordinate) in that order;
  * Eq. 1 is taken literally: frequencies 2^l with no factor pi, feature order
    [x, sin(2^0 x), cos(2^0 x), ..., sin(2^(L-1) x), cos(2^(L-1) x)], each block 2 wide.
"""
from __future__ import annotations

import numpy as np


def coordinates(window: int) -> np.ndarray:
    """x in [-1, 1]^(n x 2): row and column coordinate of token i = y * window + x."""
    lin = np.zeros(1) if window == 1 else np.linspace(-1.0, 1.0, window)
    yy, xx = np.meshgrid(lin, lin, indexing="ij")
    return np.stack([yy.reshape(-1), xx.reshape(-1)], axis=1)


def fourier_features(x: np.ndarray, L: int) -> np.ndarray:
    """Eq. 1: r_in = gamma(x), shape [n, 2 + 4 L]."""
    blocks = [x]
    for l in range(L):
        blocks.append(np.sin((2.0 ** l) * x))
        blocks.append(np.cos((2.0 ** l) * x))
    return np.concatenate(blocks, axis=1)


def forward(w_h, b_h, w_pq, w_pk, window: int, L: int):
    """Eq. 2 and Eq. 3: returns (Pq [n, R], Pk [n, R], h [n, d_h], r_in [n, 2 + 4 L]) in float64."""
    w_h, b_h, w_pq, w_pk = (np.asarray(a, dtype=np.float64) for a in (w_h, b_h, w_pq, w_pk))
    r_in = fourier_features(coordinates(window), L)
    h = np.maximum(r_in @ w_h + b_h, 0.0)          # Eq. 2
    return h @ w_pq, h @ w_pk, h, r_in             # Eq. 3


def backward(w_h, b_h, w_pq, w_pk, dpq, dpk, window: int, L: int):
    """Gradients of sum(Pq * dpq) + sum(Pk * dpk) with respect to W_h, b_h, W_pq, W_pk."""
    w_h, b_h, w_pq, w_pk, dpq, dpk = (np.asarray(a, dtype=np.float64) for a in (w_h, b_h, w_pq, w_pk, dpq, dpk))
    _, _, h, r_in = forward(w_h, b_h, w_pq, w_pk, window, L)
    dw_pq = h.T @ dpq
    dw_pk = h.T @ dpk
    dh = dpq @ w_pq.T + dpk @ w_pk.T
    da = dh * (h > 0.0)                            # through the ReLU of Eq. 2
    return r_in.T @ da, da.sum(axis=0), dw_pq, dw_pk

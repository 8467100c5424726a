"""CPU oracle for the Convolutional Local Attention gate (Sec. 3.2, Eq. 8 and Eq. 9).

TEST INFRASTRUCTURE ONLY: plain numpy in float64, written from the paper's equations; it shares no
code with the CUDA path.  Only tests, the smoke check and the benchmark's CPU leg may import it.

Eq. 8:  G~ = sigmoid(PWConv(DWConv3x3(F^-1(X))))   on the H x W x D feature map of the tokens X
Eq. 9:  O' = O o G,  G = F(G~)                       (element-wise product with the attention output)

F and F^-1 only reshape between the token list and the 2-D map (Eq. 7); with tensors kept as
[B, H, W, D] they are the identity here.  Readings where the paper is silent (parity unpinned
against the paper, which prints no example):
  * DWConv3x3: one 3 x 3 filter per channel, stride 1, zero padding 1, with a bias per channel;
    w_dw[c, dy, dx] multiplies X[y + dy - 1, x + dx - 1, c] (cross-correlation, as deep-learning
    libraries define convolution);
  * PWConv: a 1 x 1 convolution, i.e. a D x D matrix over channels, w_pw[out, in], with a bias.
"""
from __future__ import annotations

import numpy as np


def dwconv3x3(x, w_dw, b_dw):
    """x [B,H,W,D], w_dw [D,3,3], b_dw [D] -> [B,H,W,D]."""
    x = np.asarray(x, dtype=np.float64)
    w_dw = np.asarray(w_dw, dtype=np.float64)
    B, H, W, D = x.shape
    xp = np.zeros((B, H + 2, W + 2, D))
    xp[:, 1:H + 1, 1:W + 1] = x
    y = np.broadcast_to(np.asarray(b_dw, dtype=np.float64), x.shape).copy()
    for dy in range(3):
        for dx in range(3):
            y += xp[:, dy:dy + H, dx:dx + W, :] * w_dw[:, dy, dx]
    return y


def pwconv(y, w_pw, b_pw):
    """y [B,H,W,D], w_pw [Dout, Din], b_pw [Dout] -> [B,H,W,Dout]."""
    return np.asarray(y, dtype=np.float64) @ np.asarray(w_pw, dtype=np.float64).T + np.asarray(b_pw, dtype=np.float64)


def gate(x, w_dw, b_dw, w_pw, b_pw):
    """Eq. 8: the gate G~ in (0, 1), [B,H,W,D]."""
    z = pwconv(dwconv3x3(x, w_dw, b_dw), w_pw, b_pw)
    return 1.0 / (1.0 + np.exp(-z))


def gated_output(out, g):
    """Eq. 9: O' = O o G; out [B,H,W,heads,d], g [B,H,W,heads*d]."""
    out = np.asarray(out, dtype=np.float64)
    return out * np.asarray(g, dtype=np.float64).reshape(out.shape)

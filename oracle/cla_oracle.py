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


def gated_output_bwd(out, g, dout_gated):
    """Chain rule of Eq. 9: (dO, dG) = (dO' o G, dO' o O), dG in the gate's [B,H,W,heads*d] layout."""
    out = np.asarray(out, dtype=np.float64)
    g = np.asarray(g, dtype=np.float64)
    dgo = np.asarray(dout_gated, dtype=np.float64)
    return dgo * g.reshape(out.shape), (dgo * out).reshape(g.shape)


def gate_bwd(x, w_dw, b_dw, w_pw, b_pw, dgate):
    """Chain rule of Eq. 8 for a gradient dgate [B,H,W,D] on the gate.

    With Y = DWConv3x3(X), Z = PWConv(Y), G = sigmoid(Z):
        dZ = dG o G o (1 - G);       db_pw[o] = sum_pixels dZ[o];   dw_pw[o, i] = sum_pixels dZ[o] Y[i];
        dY[i] = sum_o dZ[o] w_pw[o, i];                             db_dw[c] = sum_pixels dY[c];
        dw_dw[c, dy, dx] = sum_pixels dY[y, x, c] X[y + dy - 1, x + dx - 1, c]   (zero outside the map);
        dX[y, x, c] = sum_{dy, dx} dY[y - dy + 1, x - dx + 1, c] w_dw[c, dy, dx]  (zero outside the map).
    Returns dx [B,H,W,D], dw_dw [D,3,3], db_dw [D], dw_pw [D,D], db_pw [D].
    """
    x = np.asarray(x, dtype=np.float64)
    w_dw = np.asarray(w_dw, dtype=np.float64)
    w_pw = np.asarray(w_pw, dtype=np.float64)
    dgate = np.asarray(dgate, dtype=np.float64)
    B, H, W, D = x.shape
    y = dwconv3x3(x, w_dw, b_dw)
    g = 1.0 / (1.0 + np.exp(-pwconv(y, w_pw, b_pw)))
    dz = dgate * g * (1.0 - g)
    db_pw = dz.sum(axis=(0, 1, 2))
    dw_pw = dz.reshape(-1, D).T @ y.reshape(-1, D)
    dy = dz @ w_pw
    db_dw = dy.sum(axis=(0, 1, 2))
    xp = np.zeros((B, H + 2, W + 2, D))
    xp[:, 1:H + 1, 1:W + 1] = x
    dyp = np.zeros((B, H + 2, W + 2, D))
    dyp[:, 1:H + 1, 1:W + 1] = dy
    dw_dw = np.zeros((D, 3, 3))
    dx = np.zeros(x.shape)
    for ky in range(3):
        for kx in range(3):
            dw_dw[:, ky, kx] = (dy * xp[:, ky:ky + H, kx:kx + W, :]).sum(axis=(0, 1, 2))
            dx += dyp[:, 2 - ky:2 - ky + H, 2 - kx:2 - kx + W, :] * w_dw[:, ky, kx]
    return dx, dw_dw, db_dw, dw_pw, db_pw

"""CPU oracle for RIB window attention on feature maps whose sides are not multiples of the window.

TEST INFRASTRUCTURE ONLY.  Plain numpy in float64, written from the paper; it shares no code with
the CUDA path nor with the C oracle of the divisible case (which serves as one of its pins).  Only
tests, the smoke check and the benchmark's CPU leg may import it.

What it computes.  The paper cuts a feature map into M x M windows and, where the map is smaller
than a multiple of the window, pads it up to one (Sec. 4, the remark that a 96 x 96 window on
64 x 64 training patches would need a lot of padding); it does not say what the padded positions
do inside the attention.  Reading taken here (parity unpinned against the paper for lack of a
printed example): the map is extended at the bottom and the right to Hp = ceil(H / M) M and
Wp = ceil(W / M) M, windows (and the cyclic shift, if any) are laid over the extended map, and
the added positions are not tokens: they are neither attended to nor produce an output.  Inside
every window the logits of Eq. 6, SoftMax and O = P V (Sec. 2.2, Sec. 3.1) run over the real
tokens of that window only, each keeping the positional row i = y M + x of its place in the
window.  For H and W multiples of M this is the divisible case unchanged.
"""
from __future__ import annotations

import numpy as np


def padded_size(H: int, W: int, window: int) -> tuple[int, int]:
    """Sides of the extended map: the next multiples of the window."""
    return -(-H // window) * window, -(-W // window) * window


def window_tokens(H, W, window, shift, wy, wx):
    """For window (wy, wx): the positional rows i of its real tokens and their pixels (Y, X)."""
    Hp, Wp = padded_size(H, W, window)
    rows, ys, xs = [], [], []
    for y in range(window):
        for x in range(window):
            Y = (wy * window + y + shift) % Hp
            X = (wx * window + x + shift) % Wp
            if Y < H and X < W:
                rows.append(y * window + x)
                ys.append(Y)
                xs.append(X)
    return np.array(rows, dtype=np.int64), np.array(ys, dtype=np.int64), np.array(xs, dtype=np.int64)


def fwd(q, k, v, pq, pk, window, shift=0):
    """out [B,H,W,heads,d] and lse [B,heads,H,W] in float64.

    q, k, v: [B,H,W,heads,d] with any positive H, W; pq, pk: [n,r] or [heads,n,r], n = window^2.
    """
    q = np.asarray(q, dtype=np.float64)
    k = np.asarray(k, dtype=np.float64)
    v = np.asarray(v, dtype=np.float64)
    pq = np.asarray(pq, dtype=np.float64)
    pk = np.asarray(pk, dtype=np.float64)
    B, H, W, heads, d = q.shape
    r = pq.shape[-1]
    if not 0 <= shift < window:
        raise ValueError("shift must lie in [0, window)")
    Hp, Wp = padded_size(H, W, window)
    out = np.full(q.shape, np.nan)
    lse = np.full((B, heads, H, W), np.nan)
    for wy in range(Hp // window):
        for wx in range(Wp // window):
            rows, ys, xs = window_tokens(H, W, window, shift, wy, wx)
            if rows.size == 0:
                continue
            for h in range(heads):
                pqh = pq[h] if pq.ndim == 3 else pq
                pkh = pk[h] if pk.ndim == 3 else pk
                bias = pqh[rows] @ pkh[rows].T / np.sqrt(r) if r else 0.0
                for b in range(B):
                    qw, kw, vw = q[b, ys, xs, h], k[b, ys, xs, h], v[b, ys, xs, h]
                    s = qw @ kw.T / np.sqrt(d) + bias                     # Eq. 6
                    mx = s.max(axis=1, keepdims=True)
                    e = np.exp(s - mx)
                    den = e.sum(axis=1, keepdims=True)
                    out[b, ys, xs, h] = (e / den) @ vw
                    lse[b, h, ys, xs] = (mx + np.log(den))[:, 0]
    return out, lse


def bwd(q, k, v, pq, pk, dout, window, shift=0):
    """dq, dk, dv [B,H,W,heads,d] and dpq, dpk (shape of pq) in float64: the chain rule of `fwd`.

    Per window and head, over the real tokens only (P, S as in `fwd`):
        dV = P^T dO;  dP = dO V^T;  dS = P o (dP - rowsum(dP o P));
        dq = dS k / sqrt(d);  dk = dS^T q / sqrt(d);
        dPq[rows] += dS Pk[rows] / sqrt(r);  dPk[rows] += dS^T Pq[rows] / sqrt(r),
    the last two summed over batch items and windows (and over heads when the table is shared).
    """
    q = np.asarray(q, dtype=np.float64)
    k = np.asarray(k, dtype=np.float64)
    v = np.asarray(v, dtype=np.float64)
    dout = np.asarray(dout, dtype=np.float64)
    pq = np.asarray(pq, dtype=np.float64)
    pk = np.asarray(pk, dtype=np.float64)
    B, H, W, heads, d = q.shape
    r = pq.shape[-1]
    if not 0 <= shift < window:
        raise ValueError("shift must lie in [0, window)")
    Hp, Wp = padded_size(H, W, window)
    dq, dk, dv = (np.full(q.shape, np.nan) for _ in range(3))
    dpq, dpk = np.zeros(pq.shape), np.zeros(pk.shape)
    for wy in range(Hp // window):
        for wx in range(Wp // window):
            rows, ys, xs = window_tokens(H, W, window, shift, wy, wx)
            if rows.size == 0:
                continue
            for h in range(heads):
                pqh = pq[h] if pq.ndim == 3 else pq
                pkh = pk[h] if pk.ndim == 3 else pk
                gq = dpq[h] if pq.ndim == 3 else dpq
                gk = dpk[h] if pk.ndim == 3 else dpk
                bias = pqh[rows] @ pkh[rows].T / np.sqrt(r) if r else 0.0
                for b in range(B):
                    qw, kw, vw, go = q[b, ys, xs, h], k[b, ys, xs, h], v[b, ys, xs, h], dout[b, ys, xs, h]
                    s = qw @ kw.T / np.sqrt(d) + bias
                    e = np.exp(s - s.max(axis=1, keepdims=True))
                    p = e / e.sum(axis=1, keepdims=True)
                    dp = go @ vw.T
                    ds = p * (dp - (dp * p).sum(axis=1, keepdims=True))
                    dv[b, ys, xs, h] = p.T @ go
                    dq[b, ys, xs, h] = ds @ kw / np.sqrt(d)
                    dk[b, ys, xs, h] = ds.T @ qw / np.sqrt(d)
                    if r:
                        np.add.at(gq, rows, ds @ pkh[rows] / np.sqrt(r))
                        np.add.at(gk, rows, ds.T @ pqh[rows] / np.sqrt(r))
    return dq, dk, dv, dpq, dpk

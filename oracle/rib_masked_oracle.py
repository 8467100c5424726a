"""CPU oracle for RIB window attention with shifted windows whose wrapped parts do not attend to each other.

TEST INFRASTRUCTURE ONLY.  Plain numpy in float64; it shares no code with the CUDA path nor with the other
oracles (the C oracle of the unmasked case serves as one of its pins).  Only tests, the smoke check and the
benchmark's CPU leg may import it.

What it computes.  The paper replaces shifted windows by a cycle of window sizes (Sec. 3.3) and defines no
shift; the benchmark configurations add a cyclic shift: the map is rolled by (-s, -s), cut into M x M windows,
attended, and rolled back, so a window in the last window row (column) holds tokens from the bottom (right) and,
wrapped around, from the top (left) of the map.  The unmasked entry points let those attend to each other.
This oracle is the usual shifted-window alternative: in the rolled frame (row Yr = wy M + y, column Xr likewise)
every token gets a region label

    ry = 0 if Yr < H - M,   1 if H - M <= Yr < H - s,   2 if Yr >= H - s        (rx likewise with W),

and inside a window a query attends only to the keys with its own (ry, rx); every other logit of Eq. 6 is
minus infinity before the SoftMax.  With s = 0 no window holds two labels and this is the unmasked case.
Parity unpinned against the paper (it has no shift); pinned against the C oracle at s = 0, against masked
library attention on an explicitly rolled map with a label image painted by slices, and by invariance tests.
"""
from __future__ import annotations

import numpy as np


def region_labels(H: int, W: int, window: int, shift: int) -> np.ndarray:
    """Label 3 ry + rx of every position (Yr, Xr) of the rolled frame, shape [H, W]."""
    def axis(n):
        t = np.arange(n)
        return np.where(t < n - window, 0, np.where(t < n - shift, 1, 2))
    return 3 * axis(H)[:, None] + axis(W)[None, :]


def _window(H, W, window, shift, wy, wx):
    """Rolled-frame and image coordinates of the tokens of window (wy, wx), in row order i = y M + x."""
    y, x = np.divmod(np.arange(window * window), window)
    Yr, Xr = wy * window + y, wx * window + x
    return Yr, Xr, (Yr + shift) % H, (Xr + shift) % W


def _check(q, window, shift):
    B, H, W, heads, d = q.shape
    if H % window or W % window:
        raise ValueError("the masked case is defined on maps that are multiples of the window")
    if not 0 <= shift < window:
        raise ValueError("shift must lie in [0, window)")
    return B, H, W, heads, d


def fwd(q, k, v, pq, pk, window, shift=0):
    """out [B,H,W,heads,d] and lse [B,heads,H,W] in float64; pq, pk: [n,r] or [heads,n,r]."""
    q, k, v, pq, pk = (np.asarray(a, dtype=np.float64) for a in (q, k, v, pq, pk))
    B, H, W, heads, d = _check(q, window, shift)
    r = pq.shape[-1]
    labels = region_labels(H, W, window, shift)
    out = np.full(q.shape, np.nan)
    lse = np.full((B, heads, H, W), np.nan)
    for wy in range(H // window):
        for wx in range(W // window):
            Yr, Xr, ys, xs = _window(H, W, window, shift, wy, wx)
            lab = labels[Yr, Xr]
            allowed = lab[:, None] == lab[None, :]
            for h in range(heads):
                pqh = pq[h] if pq.ndim == 3 else pq
                pkh = pk[h] if pk.ndim == 3 else pk
                bias = pqh @ pkh.T / np.sqrt(r) if r else 0.0
                for b in range(B):
                    qw, kw, vw = q[b, ys, xs, h], k[b, ys, xs, h], v[b, ys, xs, h]
                    s = np.where(allowed, qw @ kw.T / np.sqrt(d) + bias, -np.inf)        # Eq. 6, then the mask
                    mx = s.max(axis=1, keepdims=True)
                    e = np.exp(s - mx)
                    den = e.sum(axis=1, keepdims=True)
                    out[b, ys, xs, h] = (e / den) @ vw
                    lse[b, h, ys, xs] = (mx + np.log(den))[:, 0]
    return out, lse


def bwd(q, k, v, pq, pk, dout, window, shift=0):
    """dq, dk, dv [B,H,W,heads,d] and dpq, dpk (shape of pq) in float64: the chain rule of `fwd`.

    A masked logit is a constant, so its P and dS are zero; otherwise as in the unmasked case:
        dV = P^T dO;  dP = dO V^T;  dS = P o (dP - rowsum(dP o P));
        dq = dS k / sqrt(d);  dk = dS^T q / sqrt(d);  dPq += dS Pk / sqrt(r);  dPk += dS^T Pq / sqrt(r).
    """
    q, k, v, pq, pk, dout = (np.asarray(a, dtype=np.float64) for a in (q, k, v, pq, pk, dout))
    B, H, W, heads, d = _check(q, window, shift)
    r = pq.shape[-1]
    labels = region_labels(H, W, window, shift)
    dq, dk, dv = (np.full(q.shape, np.nan) for _ in range(3))
    dpq, dpk = np.zeros(pq.shape), np.zeros(pk.shape)
    for wy in range(H // window):
        for wx in range(W // window):
            Yr, Xr, ys, xs = _window(H, W, window, shift, wy, wx)
            lab = labels[Yr, Xr]
            allowed = lab[:, None] == lab[None, :]
            for h in range(heads):
                pqh = pq[h] if pq.ndim == 3 else pq
                pkh = pk[h] if pk.ndim == 3 else pk
                gq = dpq[h] if pq.ndim == 3 else dpq
                gk = dpk[h] if pk.ndim == 3 else dpk
                bias = pqh @ pkh.T / np.sqrt(r) if r else 0.0
                for b in range(B):
                    qw, kw, vw, go = q[b, ys, xs, h], k[b, ys, xs, h], v[b, ys, xs, h], dout[b, ys, xs, h]
                    s = np.where(allowed, qw @ kw.T / np.sqrt(d) + bias, -np.inf)
                    e = np.exp(s - s.max(axis=1, keepdims=True))
                    p = e / e.sum(axis=1, keepdims=True)
                    dp = go @ vw.T
                    ds = p * (dp - (dp * p).sum(axis=1, keepdims=True))
                    dv[b, ys, xs, h] = p.T @ go
                    dq[b, ys, xs, h] = ds @ kw / np.sqrt(d)
                    dk[b, ys, xs, h] = ds.T @ qw / np.sqrt(d)
                    if r:
                        gq += ds @ pkh / np.sqrt(r)
                        gk += ds.T @ pqh / np.sqrt(r)
    return dq, dk, dv, dpq, dpk

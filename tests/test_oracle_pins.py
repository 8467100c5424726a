"""Pins for the CPU oracle: each test checks it against something other than itself.

The independent routes used here: an explicit additive-bias formulation with numpy roll/reshape
window partitioning (Eq. 6 read right to left), torch's CPU scaled-dot-product attention, closed
forms, pure-Python brute force, central finite differences, and structural invariants.
"""
import itertools
import math
from pathlib import Path

import numpy as np
import pytest
import torch

from oracle import rib_oracle as orc

GOLDEN = Path(__file__).parent / "golden"


def rand_case(rng, B, H, W, heads, d, r, window, headwise=False, sigma_p=0.5):
    n = window * window
    q, k, v = (rng.standard_normal((B, H, W, heads, d)) for _ in range(3))
    pshape = (heads, n, r) if headwise else (n, r)
    pq, pk = (sigma_p * rng.standard_normal(pshape) for _ in range(2))
    return q, k, v, pq, pk


def partition(x, window, shift):
    """[B,H,W,heads,d] -> [B,nWy,nWx,heads,n,d] by roll + reshape (not the oracle's index formula)."""
    B, H, W, heads, d = x.shape
    x = np.roll(x, (-shift, -shift), axis=(1, 2))
    x = x.reshape(B, H // window, window, W // window, window, heads, d)
    return x.transpose(0, 1, 3, 5, 2, 4, 6).reshape(B, H // window, W // window, heads, window * window, d)


def unpartition(xw, H, W, window, shift):
    B, nWy, nWx, heads, n, d = xw.shape
    x = xw.reshape(B, nWy, nWx, heads, window, window, d).transpose(0, 1, 4, 2, 5, 3, 6)
    x = x.reshape(B, H, W, heads, d)
    return np.roll(x, (shift, shift), axis=(1, 2))


def additive_bias_attention(q, k, v, pq, pk, window, shift):
    """softmax(q k^T / sqrt(d) + Bias) v with Bias = pq pk^T / sqrt(r) materialised (n x n)."""
    B, H, W, heads, d = q.shape
    r = pq.shape[-1]
    qw, kw, vw = (partition(t, window, shift) for t in (q, k, v))
    bias = pq @ np.swapaxes(pk, -1, -2) / math.sqrt(r) if r else np.zeros((window ** 2,) * 2)
    if bias.ndim == 3:  # head-wise
        bias = bias[None, None, None]
    S = qw @ np.swapaxes(kw, -1, -2) / math.sqrt(d) + bias
    mx = S.max(-1, keepdims=True)
    E = np.exp(S - mx)
    den = E.sum(-1, keepdims=True)
    out = unpartition((E / den) @ vw, H, W, window, shift)
    lse_w = (mx + np.log(den))[..., 0]                                   # [B,nWy,nWx,heads,n]
    lse = unpartition(lse_w[..., None], H, W, window, shift)[..., 0]     # [B,H,W,heads]
    return out, lse.transpose(0, 3, 1, 2)


CASES = [  # B, H, W, heads, d, r, window, shift
    (1, 4, 4, 1, 2, 1, 2, 0),
    (2, 8, 8, 2, 4, 2, 4, 2),
    (1, 8, 12, 3, 8, 4, 4, 1),
    (2, 16, 16, 2, 32, 16, 8, 4),
    (1, 12, 6, 2, 5, 3, 6, 5),
    (1, 16, 32, 2, 32, 16, 16, 8),
]


@pytest.mark.parametrize("case", CASES)
@pytest.mark.parametrize("headwise", [False, True])
def test_concat_form_equals_additive_bias(case, headwise):
    """Eq. 6: the concatenated dot product equals content/sqrt(d) + materialised bias/sqrt(r)."""
    B, H, W, heads, d, r, window, shift = case
    rng = np.random.default_rng(hash(case) % 2**32)
    q, k, v, pq, pk = rand_case(rng, B, H, W, heads, d, r, window, headwise)
    out, lse = orc.fwd(q, k, v, pq, pk, window, shift)
    ref_out, ref_lse = additive_bias_attention(q, k, v, pq, pk, window, shift)
    np.testing.assert_allclose(out, ref_out, rtol=0, atol=1e-12)
    np.testing.assert_allclose(lse, ref_lse, rtol=0, atol=1e-12)


def test_zero_bias_reduces_to_library_sdpa():
    """With Pq = Pk = 0 the method is standard attention: compare with torch's CPU SDPA."""
    B, H, W, heads, d, r, window, shift = 2, 8, 8, 2, 16, 4, 4, 2
    rng = np.random.default_rng(7)
    q, k, v, pq, pk = rand_case(rng, B, H, W, heads, d, r, window)
    out, _ = orc.fwd(q, k, v, 0 * pq, 0 * pk, window, shift)
    qw, kw, vw = (torch.from_numpy(partition(t, window, shift)) for t in (q, k, v))
    ref = torch.nn.functional.scaled_dot_product_attention(qw, kw, vw)  # scale 1/sqrt(d)
    np.testing.assert_allclose(out, unpartition(ref.numpy(), H, W, window, shift), atol=1e-12)


def test_rank_zero_is_plain_attention():
    B, H, W, heads, d, window, shift = 1, 8, 8, 2, 8, 4, 1
    rng = np.random.default_rng(8)
    q, k, v, _, _ = rand_case(rng, B, H, W, heads, d, 1, window)
    empty = np.zeros((window * window, 0))
    out, _ = orc.fwd(q, k, v, empty, empty, window, shift)
    qw, kw, vw = (torch.from_numpy(partition(t, window, shift)) for t in (q, k, v))
    ref = torch.nn.functional.scaled_dot_product_attention(qw, kw, vw)
    np.testing.assert_allclose(out, unpartition(ref.numpy(), H, W, window, shift), atol=1e-12)


def test_bias_only_changes_result():
    """The bias term is really used: a non-zero Pq, Pk moves the output."""
    rng = np.random.default_rng(9)
    q, k, v, pq, pk = rand_case(rng, 1, 8, 8, 1, 8, 4, 4)
    a, _ = orc.fwd(q, k, v, pq, pk, 4, 0)
    b, _ = orc.fwd(q, k, v, 0 * pq, pk, 4, 0)
    assert np.abs(a - b).max() > 1e-3


def test_uniform_attention_closed_form():
    """q = 0 and Pq = 0 give S = 0: every output is the window mean of v and lse = ln n."""
    B, H, W, heads, d, r, window, shift = 1, 8, 8, 2, 4, 2, 4, 3
    rng = np.random.default_rng(10)
    q, k, v, pq, pk = rand_case(rng, B, H, W, heads, d, r, window)
    out, lse = orc.fwd(0 * q, k, v, 0 * pq, pk, window, shift)
    mean = partition(v, window, shift).mean(axis=4, keepdims=True)
    ref = unpartition(np.broadcast_to(mean, partition(v, window, shift).shape).copy(), H, W, window, shift)
    np.testing.assert_allclose(out, ref, atol=1e-13)
    np.testing.assert_allclose(lse, math.log(window * window), atol=1e-13)


def test_single_token_window_returns_v():
    rng = np.random.default_rng(11)
    q, k, v, pq, pk = rand_case(rng, 2, 3, 5, 2, 4, 3, 1)
    out, lse = orc.fwd(q, k, v, pq, pk, 1, 0)
    np.testing.assert_allclose(out, v, atol=0)
    s = (q * k).sum(-1) / 2.0 + (pq[0] * pk[0]).sum() / math.sqrt(3)
    np.testing.assert_allclose(lse, s.transpose(0, 3, 1, 2), atol=1e-13)


def test_toy_repeated_pattern_closed_form():
    """Fig. 1(b) toy: a 32x32 map tiling two orthogonal 32-d vectors, Q = K, no positional term.

    Attention then depends on content equality only (the checkerboard): with |a|^2 = |b|^2 = alpha,
    p_same / p_diff = exp(alpha / sqrt(d)), rows sum to one, lse = ln((n/2)(e^{alpha/sqrt d} + 1)).
    Expected values come from tests/golden/toy_checkerboard.txt (written from the closed form).
    """
    vals = dict(line.split("=") for line in (GOLDEN / "toy_checkerboard.txt").read_text().splitlines()
                if line and not line.startswith("#"))
    M, d, alpha = int(vals["M"]), int(vals["d"]), float(vals["alpha"])
    a = np.zeros(d); a[: d // 2] = math.sqrt(alpha / (d // 2))
    b = np.zeros(d); b[d // 2:] = math.sqrt(alpha / (d // 2))
    yy, xx = np.mgrid[0:M, 0:M]
    kind = (yy + xx) % 2                                      # checkerboard tiling
    x = np.where(kind[..., None] == 0, a, b)[None, :, :, None, :]   # [1,M,M,1,d]
    v = np.zeros((1, M, M, 1, d)); v[0, :, :, 0, 0] = (kind == 0); v[0, :, :, 0, 1] = (kind == 1)
    z = np.zeros((M * M, 4))
    out, lse = orc.fwd(x, x, v, z, z, M, 0)
    p_same_total, p_diff_total, ref_lse = (float(vals[s]) for s in ("p_same_total", "p_diff_total", "lse"))
    same = np.where(kind == 0, out[0, :, :, 0, 0], out[0, :, :, 0, 1])
    diff = np.where(kind == 0, out[0, :, :, 0, 1], out[0, :, :, 0, 0])
    np.testing.assert_allclose(same, p_same_total, rtol=1e-12)
    np.testing.assert_allclose(diff, p_diff_total, rtol=1e-12)
    np.testing.assert_allclose(lse, ref_lse, rtol=1e-13)
    P, _ = orc.pair_matrices(x, x, v, z, z, None, M, 0, 0)
    np.testing.assert_allclose(P[0, 2] / P[0, 1], math.exp(alpha / math.sqrt(d)), rtol=1e-12)


def brute_force(q, k, v, pq, pk, window, shift):
    """Loop-only transcription of Eq. 5: build the concatenated rows, one dot product, no max trick."""
    B, H, W, heads, d = q.shape
    n, r = pq.shape
    out = np.zeros_like(q)
    for b, wy, wx, h in itertools.product(range(B), range(H // window), range(W // window), range(heads)):
        toks = [((wy * window + y + shift) % H, (wx * window + x + shift) % W)
                for y in range(window) for x in range(window)]
        Qt = [list(q[b, Y, X, h] / math.sqrt(d)) + list(pq[i] / math.sqrt(r)) for i, (Y, X) in enumerate(toks)]
        Kt = [list(k[b, Y, X, h]) + list(pk[i]) for i, (Y, X) in enumerate(toks)]
        for i, (Y, X) in enumerate(toks):
            e = [math.exp(sum(a * c for a, c in zip(Qt[i], Kt[j]))) for j in range(n)]
            tot = sum(e)
            for c in range(d):
                out[b, Y, X, h, c] = sum(e[j] / tot * v[b, toks[j][0], toks[j][1], h, c] for j in range(n))
    return out


@pytest.mark.parametrize("case", [(1, 4, 4, 1, 2, 1, 2, 0), (2, 8, 8, 2, 4, 2, 4, 2), (1, 4, 6, 2, 3, 2, 2, 1)])
def test_brute_force_tiny(case):
    B, H, W, heads, d, r, window, shift = case
    rng = np.random.default_rng(12)
    q, k, v, pq, pk = rand_case(rng, B, H, W, heads, d, r, window)
    out, _ = orc.fwd(q, k, v, pq, pk, window, shift)
    np.testing.assert_allclose(out, brute_force(q, k, v, pq, pk, window, shift), atol=1e-12)


def test_softmax_rows_sum_to_one_and_match_lse():
    rng = np.random.default_rng(13)
    q, k, v, pq, pk = rand_case(rng, 1, 8, 8, 2, 8, 4, 4)
    for pid in range(orc.num_pairs(1, 8, 8, 2, 4)):
        P, _ = orc.pair_matrices(q, k, v, pq, pk, None, 4, 2, pid)
        np.testing.assert_allclose(P.sum(1), 1.0, atol=1e-13)
        assert (P > 0).all()


@pytest.mark.parametrize("H,W,window,shift", [(8, 8, 4, 0), (8, 8, 4, 2), (12, 6, 6, 5), (16, 32, 16, 8),
                                             (96, 96, 48, 24), (6, 9, 3, 1)])
def test_partition_and_shift_are_bijections(H, W, window, shift):
    """Every pixel belongs to exactly one (window, token); the map matches roll + reshape."""
    ids = np.arange(H * W).reshape(1, H, W, 1, 1).astype(float)
    seen = np.zeros((H, W), dtype=int)
    parted = partition(ids, window, shift)
    for wy in range(H // window):
        for wx in range(W // window):
            for i in range(window * window):
                Y, X = orc.token_pixel(H, W, window, shift, wy, wx, i)
                seen[Y, X] += 1
                assert parted[0, wy, wx, 0, i, 0] == Y * W + X
    assert (seen == 1).all()
    np.testing.assert_array_equal(unpartition(parted, H, W, window, shift), ids)
    if shift == 0:
        assert orc.token_pixel(H, W, window, 0, 0, 0, window + 1) == (1, 1)


def test_shift_equals_rolled_input():
    """Attention with shift s on x equals attention with shift 0 on x rolled by -s, rolled back."""
    rng = np.random.default_rng(14)
    q, k, v, pq, pk = rand_case(rng, 1, 8, 8, 2, 4, 2, 4)
    s = 3
    out_s, lse_s = orc.fwd(q, k, v, pq, pk, 4, s)
    rq, rk, rv = (np.roll(t, (-s, -s), axis=(1, 2)) for t in (q, k, v))
    out_0, lse_0 = orc.fwd(rq, rk, rv, pq, pk, 4, 0)
    np.testing.assert_allclose(out_s, np.roll(out_0, (s, s), axis=(1, 2)), atol=1e-14)
    np.testing.assert_allclose(lse_s, np.roll(lse_0, (s, s), axis=(2, 3)), atol=1e-14)


def test_windows_share_the_bias_and_are_independent():
    """Swapping two windows' contents swaps their outputs (same Pq/Pk everywhere, no leakage)."""
    rng = np.random.default_rng(15)
    q, k, v, pq, pk = rand_case(rng, 1, 8, 8, 1, 4, 2, 4)
    out, _ = orc.fwd(q, k, v, pq, pk, 4, 0)

    def swap(t):
        t = t.copy()
        t[:, 0:4, 0:4], t[:, 4:8, 4:8] = t[:, 4:8, 4:8].copy(), t[:, 0:4, 0:4].copy()
        return t

    out2, _ = orc.fwd(swap(q), swap(k), swap(v), pq, pk, 4, 0)
    np.testing.assert_allclose(out2, swap(out), atol=1e-14)


def test_token_permutation_equivariance():
    """Permuting tokens inside a window together with their Pq/Pk rows permutes the output."""
    rng = np.random.default_rng(16)
    M = 4
    q, k, v, pq, pk = rand_case(rng, 1, M, M, 1, 4, 2, M)
    perm = rng.permutation(M * M)
    out, _ = orc.fwd(q, k, v, pq, pk, M, 0)

    def p(t):
        return t.reshape(1, M * M, 1, -1)[:, perm].reshape(t.shape)

    out2, _ = orc.fwd(p(q), p(k), p(v), pq[perm], pk[perm], M, 0)
    np.testing.assert_allclose(out2, p(out), atol=1e-14)


def test_subset_of_pairs_matches_full_run():
    rng = np.random.default_rng(17)
    q, k, v, pq, pk = rand_case(rng, 2, 8, 8, 2, 4, 2, 4)
    full, lse = orc.fwd(q, k, v, pq, pk, 4, 1)
    part, lse_p = orc.fwd(q, k, v, pq, pk, 4, 1, pairs=[3, 10])
    mask = ~np.isnan(part)
    assert mask.sum() == 2 * 16 * 4
    np.testing.assert_array_equal(part[mask], full[mask])
    assert (~np.isnan(lse_p)).sum() == 2 * 16


# ----------------------------------------------------------------------------- backward pins

def loss(q, k, v, pq, pk, dout, window, shift):
    out, _ = orc.fwd(q, k, v, pq, pk, window, shift)
    return float((out * dout).sum())


@pytest.mark.parametrize("case", [(1, 4, 4, 1, 3, 2, 2, 1), (2, 8, 4, 2, 4, 3, 4, 2)])
@pytest.mark.parametrize("headwise", [False, True])
def test_gradients_by_central_differences(case, headwise):
    """Every gradient against a central finite difference of L = sum(out * dout) in fp64."""
    B, H, W, heads, d, r, window, shift = case
    rng = np.random.default_rng(18)
    q, k, v, pq, pk = rand_case(rng, B, H, W, heads, d, r, window, headwise)
    dout = rng.standard_normal(q.shape)
    grads = dict(zip(("q", "k", "v", "pq", "pk"), orc.bwd(q, k, v, pq, pk, dout, window, shift)))
    args = {"q": q, "k": k, "v": v, "pq": pq, "pk": pk}
    eps = 1e-5
    for name, arr in args.items():
        flat_idx = rng.choice(arr.size, size=min(arr.size, 24), replace=False)
        for fi in flat_idx:
            idx = np.unravel_index(fi, arr.shape)
            hi = {kk: vv.copy() for kk, vv in args.items()}
            lo = {kk: vv.copy() for kk, vv in args.items()}
            hi[name][idx] += eps
            lo[name][idx] -= eps
            fd = (loss(**hi, dout=dout, window=window, shift=shift)
                  - loss(**lo, dout=dout, window=window, shift=shift)) / (2 * eps)
            assert abs(fd - grads[name][idx]) <= 1e-6 * max(1.0, abs(fd)), (name, idx, fd, grads[name][idx])


def test_gradients_match_torch_autograd_of_additive_bias_form():
    """Autograd through the explicit-bias formulation (torch CPU, fp64) gives the same gradients."""
    B, H, W, heads, d, r, window, shift = 2, 8, 8, 2, 8, 4, 4, 2
    rng = np.random.default_rng(19)
    q, k, v, pq, pk = rand_case(rng, B, H, W, heads, d, r, window)
    dout = rng.standard_normal(q.shape)
    tq, tk, tv, tpq, tpk = (torch.tensor(t, requires_grad=True) for t in (q, k, v, pq, pk))

    def part(x):
        x = torch.roll(x, (-shift, -shift), dims=(1, 2))
        x = x.reshape(B, H // window, window, W // window, window, heads, d)
        return x.permute(0, 1, 3, 5, 2, 4, 6).reshape(B, H // window, W // window, heads, window ** 2, d)

    S = part(tq) @ part(tk).transpose(-1, -2) / math.sqrt(d) + tpq @ tpk.T / math.sqrt(r)
    O = torch.softmax(S, -1) @ part(tv)
    (O * part(torch.tensor(dout))).sum().backward()
    dq, dk, dv, dpq, dpk = orc.bwd(q, k, v, pq, pk, dout, window, shift)
    for got, ref in ((dq, tq), (dk, tk), (dv, tv), (dpq, tpq), (dpk, tpk)):
        np.testing.assert_allclose(got, ref.grad.numpy(), atol=1e-11)


def test_logit_gradient_rows_sum_to_zero():
    rng = np.random.default_rng(20)
    q, k, v, pq, pk = rand_case(rng, 1, 8, 8, 2, 4, 2, 4)
    dout = rng.standard_normal(q.shape)
    _, dS = orc.pair_matrices(q, k, v, pq, pk, dout, 4, 2, 5)
    np.testing.assert_allclose(dS.sum(1), 0.0, atol=1e-13)


def test_bias_gradient_adds_over_batch_windows_and_heads():
    """dPq of B identical images is B times dPq of one; shared Pq sums the head-wise gradients."""
    rng = np.random.default_rng(21)
    q, k, v, pq, pk = rand_case(rng, 1, 8, 8, 2, 4, 2, 4)
    dout = rng.standard_normal(q.shape)
    one = orc.bwd(q, k, v, pq, pk, dout, 4, 1)
    rep = orc.bwd(*(np.repeat(t, 3, axis=0) for t in (q, k, v)), pq, pk, np.repeat(dout, 3, axis=0), 4, 1)
    np.testing.assert_allclose(rep[3], 3 * one[3], rtol=1e-12)
    np.testing.assert_allclose(rep[4], 3 * one[4], rtol=1e-12)
    hw = orc.bwd(q, k, v, np.stack([pq, pq]), np.stack([pk, pk]), dout, 4, 1)
    np.testing.assert_allclose(hw[3].sum(0), one[3], atol=1e-12)
    np.testing.assert_allclose(hw[4].sum(0), one[4], atol=1e-12)
    # per-pair contributions add up to the full reduction
    parts = [orc.bwd(q, k, v, pq, pk, dout, 4, 1, pairs=[p]) for p in range(orc.num_pairs(1, 8, 8, 2, 4))]
    np.testing.assert_allclose(sum(p[3] for p in parts), one[3], atol=1e-12)


def test_bad_shapes_are_rejected():
    rng = np.random.default_rng(22)
    q, k, v, pq, pk = rand_case(rng, 1, 8, 8, 1, 4, 2, 4)
    with pytest.raises(ValueError):
        orc.fwd(q, k, v, pq, pk, 4, 4)          # shift must be < window
    with pytest.raises(ValueError):
        orc.fwd(q[:, :6], k[:, :6], v[:, :6], pq, pk, 4, 0)   # H not a multiple of the window

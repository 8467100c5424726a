"""Pins of the oracle for maps that are not multiples of the window (oracle/rib_padded_oracle.py):
the divisible case against the independent C oracle, the masked case against a library attention
routine on an explicitly padded and masked problem, closed forms, and planted mistakes."""
import numpy as np
import pytest
import torch

from oracle import rib_oracle as orc
from oracle import rib_padded_oracle as pad


def rand_case(seed, B, H, W, heads, d, r, window, headwise=False):
    rng = np.random.default_rng(seed)
    shape = (B, H, W, heads, d)
    q, k, v = (rng.standard_normal(shape) for _ in range(3))
    pshape = (heads, window * window, r) if headwise else (window * window, r)
    pq, pk = (0.5 * rng.standard_normal(pshape) for _ in range(2))
    return q, k, v, pq, pk


@pytest.mark.parametrize("shift", [0, 3])
@pytest.mark.parametrize("headwise", [False, True])
def test_divisible_maps_reproduce_the_c_oracle(shift, headwise):
    q, k, v, pq, pk = rand_case(1, 2, 8, 12, 2, 8, 4, 4, headwise)
    out, lse = pad.fwd(q, k, v, pq, pk, 4, shift)
    ref_out, ref_lse = orc.fwd(q, k, v, pq, pk, 4, shift)
    np.testing.assert_allclose(out, ref_out, rtol=0, atol=1e-12)
    np.testing.assert_allclose(lse, ref_lse, rtol=0, atol=1e-12)


def sdpa_reference(q, k, v, pq, pk, window, shift):
    """The same reading through a library routine: zero-extend the map, roll it, cut windows, and let
    torch's scaled_dot_product_attention apply an additive bias (the RIB logits) plus a key mask."""
    B, H, W, heads, d = q.shape
    M, n, r = window, window * window, pq.shape[-1]
    Hp, Wp = pad.padded_size(H, W, M)

    def windows(x):   # [B,H,W,heads,c] -> [B, nWy, nWx, heads, n, c] of the rolled, extended map
        ext = np.zeros((B, Hp, Wp) + x.shape[3:])
        ext[:, :H, :W] = x
        ext = np.roll(ext, (-shift, -shift), (1, 2))
        c = x.shape[-1]
        t = ext.reshape(B, Hp // M, M, Wp // M, M, heads, c).transpose(0, 1, 3, 5, 2, 4, 6)
        return t.reshape(B, Hp // M, Wp // M, heads, n, c)

    # which window positions hold real tokens: the windows of a map of ones, zero-extended like the data
    vw = windows(np.ones((B, H, W, heads, 1)))[..., 0] > 0.5                            # [B,nWy,nWx,heads,n]
    bias = pq @ pk.T / np.sqrt(r)                                                      # [n,n], shared table
    mask = np.where(vw[..., None, :], 0.0, -np.inf) + bias                              # keys masked
    qw, kw, vv = (torch.from_numpy(windows(x)) for x in (q, k, v))
    o = torch.nn.functional.scaled_dot_product_attention(qw, kw, vv, attn_mask=torch.from_numpy(mask)).numpy()
    # back to the map: undo windows, undo the roll, crop
    ext = o.reshape(B, Hp // M, Wp // M, heads, M, M, d).transpose(0, 1, 4, 2, 5, 3, 6).reshape(B, Hp, Wp, heads, d)
    ext = np.roll(ext, (shift, shift), (1, 2))
    return ext[:, :H, :W]


@pytest.mark.parametrize("H,W,window,shift", [(6, 10, 4, 0), (7, 5, 4, 1), (10, 6, 8, 3), (3, 3, 4, 0)])
def test_non_divisible_maps_against_masked_library_attention(H, W, window, shift):
    q, k, v, pq, pk = rand_case(2, 2, H, W, 2, 8, 4, window)
    out, _ = pad.fwd(q, k, v, pq, pk, window, shift)
    ref = sdpa_reference(q, k, v, pq, pk, window, shift)
    assert np.isfinite(out).all()
    np.testing.assert_allclose(out, ref, rtol=0, atol=1e-10)


def test_lse_is_the_log_of_the_softmax_denominator():
    q, k, v, pq, pk = rand_case(3, 1, 5, 7, 1, 4, 4, 4)
    out, lse = pad.fwd(q, k, v, pq, pk, 4, 0)
    # window (1, 1) of the extended 8 x 8 map holds the real pixels Y = 4, X = 4..6: three tokens
    rows, ys, xs = pad.window_tokens(5, 7, 4, 0, 1, 1)
    assert list(zip(ys, xs)) == [(4, 4), (4, 5), (4, 6)] and list(rows) == [0, 1, 2]
    s = q[0, 4, 4:7, 0] @ k[0, 4, 4:7, 0].T / 2.0 + pq[:3] @ pk[:3].T / 2.0
    np.testing.assert_allclose(lse[0, 0, 4, 4:7], np.log(np.exp(s).sum(1)), atol=1e-12)
    p = np.exp(s - lse[0, 0, 4, 4:7, None])
    np.testing.assert_allclose(out[0, 4, 4:7, 0], p @ v[0, 4, 4:7, 0], atol=1e-12)


def test_a_lone_token_returns_its_value():
    # 5 x 5 map, window 4: the extended map is 8 x 8 and window (1, 1) holds the single pixel (4, 4)
    q, k, v, pq, pk = rand_case(4, 1, 5, 5, 2, 4, 4, 4)
    out, lse = pad.fwd(q, k, v, pq, pk, 4, 0)
    np.testing.assert_allclose(out[0, 4, 4], v[0, 4, 4], atol=1e-14)
    s = (q[0, 4, 4] * k[0, 4, 4]).sum(-1) / 2.0 + (pq[0] * pk[0]).sum() / 2.0
    np.testing.assert_allclose(lse[0, :, 4, 4], s, atol=1e-14)


def test_every_real_token_is_written_exactly_once():
    for H, W, window, shift in [(6, 10, 4, 0), (7, 5, 4, 1), (9, 9, 8, 5)]:
        Hp, Wp = pad.padded_size(H, W, window)
        seen = np.zeros((H, W), dtype=int)
        for wy in range(Hp // window):
            for wx in range(Wp // window):
                _, ys, xs = pad.window_tokens(H, W, window, shift, wy, wx)
                seen[ys, xs] += 1
        assert (seen == 1).all()


def test_planted_mistakes_are_caught():
    """A wrap over the real size instead of the extended one, or padded positions treated as zero tokens,
    changes the result on a non-divisible map."""
    q, k, v, pq, pk = rand_case(5, 1, 6, 6, 1, 4, 4, 4)
    good, _ = pad.fwd(q, k, v, pq, pk, 4, 1)
    ref = sdpa_reference(q, k, v, pq, pk, 4, 1)
    np.testing.assert_allclose(good, ref, atol=1e-10)
    # mistake 1: zero tokens that take part in the softmax (no mask)
    ext = [np.pad(x, ((0, 0), (0, 2), (0, 2), (0, 0), (0, 0))) for x in (q, k, v)]
    wrong, _ = orc.fwd(np.roll(ext[0], 0, 1), ext[1], ext[2], pq, pk, 4, 1)
    assert np.abs(wrong[:, :6, :6] - good).max() > 1e-3
    # mistake 2: the cyclic shift wraps over H x W instead of Hp x Wp
    rows_good = pad.window_tokens(6, 6, 4, 1, 1, 1)
    Y_wrong = (1 * 4 + np.arange(4) + 1) % 6
    assert not np.array_equal(np.unique(rows_good[1]), np.unique(Y_wrong[Y_wrong < 6]))


# ------------------------------------------------------------------------------------------ backward
@pytest.mark.parametrize("shift", [0, 3])
@pytest.mark.parametrize("headwise", [False, True])
def test_backward_on_divisible_maps_reproduces_the_c_oracle(shift, headwise):
    q, k, v, pq, pk = rand_case(11, 2, 8, 12, 2, 8, 4, 4, headwise)
    dout = np.random.default_rng(12).standard_normal(q.shape)
    got = pad.bwd(q, k, v, pq, pk, dout, 4, shift)
    ref = orc.bwd(q, k, v, pq, pk, dout, 4, shift)
    for a, b in zip(got, ref):
        np.testing.assert_allclose(a, b, rtol=0, atol=1e-11)


@pytest.mark.parametrize("H,W,window,shift,headwise", [(6, 10, 4, 0, False), (7, 5, 4, 1, True), (3, 3, 4, 0, False)])
def test_backward_by_central_differences_on_non_divisible_maps(H, W, window, shift, headwise):
    q, k, v, pq, pk = rand_case(13, 1, H, W, 2, 4, 4, window, headwise)
    dout = np.random.default_rng(14).standard_normal(q.shape)
    grads = pad.bwd(q, k, v, pq, pk, dout, window, shift)
    assert all(np.isfinite(g).all() for g in grads)

    def loss(args):
        return float((pad.fwd(*args, window, shift)[0] * dout).sum())

    args = [q, k, v, pq, pk]
    rng = np.random.default_rng(15)
    eps = 1e-6
    for which, grad in enumerate(grads):
        x = args[which]
        for _ in range(6):
            idx = tuple(int(rng.integers(n)) for n in x.shape)
            old = x[idx]
            x[idx] = old + eps; up = loss(args)
            x[idx] = old - eps; down = loss(args)
            x[idx] = old
            np.testing.assert_allclose(grad[idx], (up - down) / (2 * eps), rtol=2e-6, atol=2e-8)


def test_backward_against_autograd_of_masked_library_attention():
    H, W, window, shift = 6, 10, 4, 1
    q, k, v, pq, pk = rand_case(16, 2, H, W, 2, 8, 4, window)
    dout = np.random.default_rng(17).standard_normal(q.shape)
    tq, tk, tv, tpq, tpk = (torch.tensor(x, requires_grad=True) for x in (q, k, v, pq, pk))
    B, _, _, heads, d = q.shape
    M, n, r = window, window * window, pq.shape[-1]
    Hp, Wp = pad.padded_size(H, W, M)

    def windows(x):
        ext = torch.zeros((B, Hp, Wp) + tuple(x.shape[3:]), dtype=x.dtype)
        ext[:, :H, :W] = x
        ext = torch.roll(ext, (-shift, -shift), (1, 2))
        c = x.shape[-1]
        return ext.reshape(B, Hp // M, M, Wp // M, M, heads, c).permute(0, 1, 3, 5, 2, 4, 6).reshape(B, Hp // M, Wp // M, heads, n, c)

    valid = windows(torch.ones((B, H, W, heads, 1), dtype=torch.float64))[..., 0] > 0.5
    mask = torch.where(valid[..., None, :], 0.0, -float("inf")) + tpq @ tpk.T / np.sqrt(r)
    o = torch.nn.functional.scaled_dot_product_attention(windows(tq), windows(tk), windows(tv), attn_mask=mask)
    ext = o.reshape(B, Hp // M, Wp // M, heads, M, M, d).permute(0, 1, 4, 2, 5, 3, 6).reshape(B, Hp, Wp, heads, d)
    out = torch.roll(ext, (shift, shift), (1, 2))[:, :H, :W]
    (out * torch.tensor(dout)).sum().backward()
    got = pad.bwd(q, k, v, pq, pk, dout, window, shift)
    for g, t in zip(got, (tq, tk, tv, tpq, tpk)):
        np.testing.assert_allclose(g, t.grad.numpy(), rtol=0, atol=1e-10)

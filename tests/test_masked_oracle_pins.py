"""Pins of the oracle for shifted windows whose wrapped parts do not attend to each other
(oracle/rib_masked_oracle.py): the unshifted case against the independent C oracle, the shifted case against a
library attention routine on an explicitly rolled map with a label image painted by slices, invariance of a
row under changes to the keys it must not see, central differences, and planted mistakes."""
import numpy as np
import pytest
import torch

from oracle import rib_masked_oracle as msk
from oracle import rib_oracle as orc


def rand_case(seed, B, H, W, heads, d, r, window, headwise=False):
    rng = np.random.default_rng(seed)
    shape = (B, H, W, heads, d)
    q, k, v = (rng.standard_normal(shape) for _ in range(3))
    pshape = (heads, window * window, r) if headwise else (window * window, r)
    pq, pk = (0.5 * rng.standard_normal(pshape) for _ in range(2))
    return q, k, v, pq, pk


def painted_labels(H, W, window, shift):
    """The label image the way shifted-window networks build it: nine rectangles of the rolled frame painted
    with consecutive numbers (a route that shares nothing with the oracle's closed form)."""
    img = np.zeros((H, W), dtype=np.int64)
    cnt = 0
    for hs in (slice(0, H - window), slice(H - window, H - shift), slice(H - shift, H)):
        for ws in (slice(0, W - window), slice(W - window, W - shift), slice(W - shift, W)):
            img[hs, ws] = cnt
            cnt += 1
    return img


def sdpa_reference(q, k, v, pq, pk, window, shift, tensors=False):
    """Roll the map, cut windows, and let torch's scaled_dot_product_attention apply the RIB logits as an
    additive bias plus minus infinity wherever the painted labels of query and key differ."""
    t = (lambda x: x) if tensors else torch.from_numpy
    B, H, W, heads, d = q.shape
    M, n, r = window, window * window, pq.shape[-1]

    def windows(x):   # [B,H,W,heads,c] -> [B, nWy, nWx, heads, n, c] of the rolled map
        x = torch.roll(x, (-shift, -shift), (1, 2))
        c = x.shape[-1]
        return x.reshape(B, H // M, M, W // M, M, heads, c).permute(0, 1, 3, 5, 2, 4, 6).reshape(B, H // M, W // M, heads, n, c)

    lab = torch.from_numpy(painted_labels(H, W, M, shift)).reshape(H // M, M, W // M, M).permute(0, 2, 1, 3).reshape(H // M, W // M, n)
    allowed = lab[..., :, None] == lab[..., None, :]                                   # [nWy, nWx, n, n]
    mask = torch.where(allowed, 0.0, -float("inf"))[None, :, :, None].to(torch.float64) + t(pq) @ t(pk).T / np.sqrt(r)
    o = torch.nn.functional.scaled_dot_product_attention(windows(t(q)), windows(t(k)), windows(t(v)), attn_mask=mask)
    o = o.reshape(B, H // M, W // M, heads, M, M, d).permute(0, 1, 4, 2, 5, 3, 6).reshape(B, H, W, heads, d)
    return torch.roll(o, (shift, shift), (1, 2))


def test_labels_equal_the_painted_rectangles_up_to_renaming():
    for H, W, M, s in [(8, 12, 4, 1), (8, 8, 8, 3), (12, 8, 4, 2), (16, 16, 8, 4)]:
        a, b = msk.region_labels(H, W, M, s), painted_labels(H, W, M, s)
        # same partition of the frame: equal labels in one image exactly where they are equal in the other
        fa, fb = a.reshape(-1), b.reshape(-1)
        assert np.array_equal(fa[:, None] == fa[None, :], fb[:, None] == fb[None, :])


@pytest.mark.parametrize("headwise", [False, True])
def test_without_a_shift_the_mask_does_nothing(headwise):
    q, k, v, pq, pk = rand_case(1, 2, 8, 12, 2, 8, 4, 4, headwise)
    out, lse = msk.fwd(q, k, v, pq, pk, 4, 0)
    ref_out, ref_lse = orc.fwd(q, k, v, pq, pk, 4, 0)
    np.testing.assert_allclose(out, ref_out, rtol=0, atol=1e-12)
    np.testing.assert_allclose(lse, ref_lse, rtol=0, atol=1e-12)
    dout = np.random.default_rng(2).standard_normal(q.shape)
    for a, b in zip(msk.bwd(q, k, v, pq, pk, dout, 4, 0), orc.bwd(q, k, v, pq, pk, dout, 4, 0)):
        np.testing.assert_allclose(a, b, rtol=0, atol=1e-11)


@pytest.mark.parametrize("H,W,window,shift", [(8, 12, 4, 1), (8, 8, 8, 3), (12, 8, 4, 2), (16, 8, 8, 4)])
def test_shifted_windows_against_masked_library_attention(H, W, window, shift):
    q, k, v, pq, pk = rand_case(3, 2, H, W, 2, 8, 4, window)
    out, _ = msk.fwd(q, k, v, pq, pk, window, shift)
    assert np.isfinite(out).all()
    np.testing.assert_allclose(out, sdpa_reference(q, k, v, pq, pk, window, shift).numpy(), rtol=0, atol=1e-10)


def test_interior_windows_equal_the_unmasked_case_and_border_windows_do_not():
    H, W, M, s = 12, 12, 4, 2
    q, k, v, pq, pk = rand_case(4, 1, H, W, 1, 4, 4, M)
    out, lse = msk.fwd(q, k, v, pq, pk, M, s)
    ref, ref_lse = orc.fwd(q, k, v, pq, pk, M, s)
    # windows 0 and 1 of the rolled frame hold one label: image rows / columns s .. 2 M + s - 1
    inner = slice(s, 2 * M + s)
    np.testing.assert_allclose(out[:, inner, inner], ref[:, inner, inner], atol=1e-12)
    np.testing.assert_allclose(lse[:, :, inner, inner], ref_lse[:, :, inner, inner], atol=1e-12)
    assert np.abs(out - ref).max() > 1e-3


def test_a_row_does_not_depend_on_the_keys_it_must_not_see():
    H, W, M, s = 8, 8, 4, 1
    q, k, v, pq, pk = rand_case(5, 1, H, W, 1, 4, 4, M)
    out, _ = msk.fwd(q, k, v, pq, pk, M, s)
    # the last window row of the rolled frame holds image rows 5, 6, 7 (label 1) and, wrapped, row 0 (label 2)
    k2, v2 = k.copy(), v.copy()
    k2[:, 0] += 3.0
    v2[:, 0] -= 2.0
    out2, _ = msk.fwd(q, k2, v2, pq, pk, M, s)
    np.testing.assert_allclose(out2[:, 1:], out[:, 1:], atol=1e-13)
    assert np.abs(out2[:, 0] - out[:, 0]).max() > 1e-2
    # the unmasked oracle does let rows 5..7 see row 0
    a, _ = orc.fwd(q, k, v, pq, pk, M, s)
    b, _ = orc.fwd(q, k2, v2, pq, pk, M, s)
    assert np.abs(a[:, 5:] - b[:, 5:]).max() > 1e-2


def test_lse_of_a_corner_region_is_the_log_sum_over_that_region_only():
    H, W, M, s = 8, 8, 4, 1
    q, k, v, pq, pk = rand_case(6, 1, H, W, 1, 4, 4, M)
    _, lse = msk.fwd(q, k, v, pq, pk, M, s)
    # the wrapped corner of the last window is the single image pixel (0, 0): window position (3, 3), row 15 of the tables
    s00 = (q[0, 0, 0, 0] * k[0, 0, 0, 0]).sum() / 2.0 + (pq[15] * pk[15]).sum() / 2.0
    np.testing.assert_allclose(lse[0, 0, 0, 0], s00, atol=1e-13)


@pytest.mark.parametrize("headwise", [False, True])
def test_backward_against_autograd_of_masked_library_attention(headwise):
    H, W, window, shift = 8, 12, 4, 1
    q, k, v, pq, pk = rand_case(7, 2, H, W, 2, 8, 4, window, headwise)
    dout = np.random.default_rng(8).standard_normal(q.shape)
    got = msk.bwd(q, k, v, pq, pk, dout, window, shift)
    if headwise:
        # one head at a time through the shared-table reference
        for h in range(2):
            ts = [torch.tensor(x, requires_grad=True) for x in (q[:, :, :, h:h + 1], k[:, :, :, h:h + 1], v[:, :, :, h:h + 1], pq[h], pk[h])]
            (sdpa_reference(*ts, window, shift, tensors=True) * torch.tensor(dout[:, :, :, h:h + 1])).sum().backward()
            for g, t, sel in zip(got, ts, (np.s_[:, :, :, h:h + 1],) * 3 + (np.s_[h],) * 2):
                np.testing.assert_allclose(g[sel], t.grad.numpy(), rtol=0, atol=1e-10)
    else:
        ts = [torch.tensor(x, requires_grad=True) for x in (q, k, v, pq, pk)]
        (sdpa_reference(*ts, window, shift, tensors=True) * torch.tensor(dout)).sum().backward()
        for g, t in zip(got, ts):
            np.testing.assert_allclose(g, t.grad.numpy(), rtol=0, atol=1e-10)


def test_backward_by_central_differences():
    H, W, window, shift = 8, 8, 4, 3
    q, k, v, pq, pk = rand_case(9, 1, H, W, 2, 4, 4, window)
    dout = np.random.default_rng(10).standard_normal(q.shape)
    grads = msk.bwd(q, k, v, pq, pk, dout, window, shift)

    def loss(args):
        return float((msk.fwd(*args, window, shift)[0] * dout).sum())

    args = [q, k, v, pq, pk]
    rng = np.random.default_rng(11)
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


def test_planted_mistakes_are_caught():
    """Labels cut at the wrong place (shift counted from the top instead of the bottom) or a mask applied to the
    rows only change the result."""
    H, W, M, s = 8, 8, 4, 1
    q, k, v, pq, pk = rand_case(12, 1, H, W, 1, 4, 4, M)
    good, _ = msk.fwd(q, k, v, pq, pk, M, s)
    np.testing.assert_allclose(good, sdpa_reference(q, k, v, pq, pk, M, s).numpy(), atol=1e-10)
    real = msk.region_labels
    try:
        msk.region_labels = lambda H_, W_, M_, s_: real(H_, W_, M_, M_ - s_)            # mistake 1
        wrong1, _ = msk.fwd(q, k, v, pq, pk, M, s)
        msk.region_labels = lambda H_, W_, M_, s_: real(H_, W_, M_, s_) // 3 * 3        # mistake 2: columns forgotten
        wrong2, _ = msk.fwd(q, k, v, pq, pk, M, s)
    finally:
        msk.region_labels = real
    assert np.abs(wrong1 - good).max() > 1e-3 and np.abs(wrong2 - good).max() > 1e-3

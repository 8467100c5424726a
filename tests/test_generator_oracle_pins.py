"""Pins of the RIB generator oracle (Eq. 1-3) against things the paper and the mathematics fix."""
import math

import numpy as np
import pytest
import torch

from oracle import rib_generator_oracle as gen


def _weights(L, dh, r, seed):
    rng = np.random.default_rng(seed)
    return (rng.normal(0, 0.5, (2 + 4 * L, dh)), rng.normal(0, 0.2, dh), rng.normal(0, 0.3, (dh, r)), rng.normal(0, 0.3, (dh, r)))


def test_embedding_width_is_2_plus_4L_and_coordinates_span_minus_one_to_one():
    for M, L in ((4, 0), (8, 3), (16, 10)):
        x = gen.coordinates(M)
        assert x.shape == (M * M, 2) and x.min() == -1.0 and x.max() == 1.0
        assert gen.fourier_features(x, L).shape == (M * M, 2 + 4 * L)      # Sec. 3.1: r_in in R^(N_w x (2 + 4L))
    assert np.array_equal(gen.coordinates(1), np.zeros((1, 2)))


def test_token_order_is_row_major():
    x = gen.coordinates(4)
    assert np.allclose(x[0], [-1, -1]) and np.allclose(x[3], [-1, 1]) and np.allclose(x[4], [-1 + 2 / 3, -1])


def test_feature_blocks_are_sines_and_cosines_of_doubling_frequencies():
    x = gen.coordinates(8)
    f = gen.fourier_features(x, 5)
    assert np.array_equal(f[:, :2], x)
    for l in range(5):
        s, c = f[:, 2 + 4 * l: 4 + 4 * l], f[:, 4 + 4 * l: 6 + 4 * l]
        assert np.allclose(s ** 2 + c ** 2, 1.0, atol=1e-14)                       # sin^2 + cos^2
        if l:
            ps, pc = f[:, 2 + 4 * (l - 1): 4 + 4 * (l - 1)], f[:, 4 + 4 * (l - 1): 6 + 4 * (l - 1)]
            assert np.allclose(s, 2 * ps * pc, atol=1e-12)                         # double-angle identities tie
            assert np.allclose(c, pc ** 2 - ps ** 2, atol=1e-12)                   # block l to block l - 1
    # scalar check of one entry, written out by hand: token (y=2, x=5) of an 8x8 window, band l = 3, column coordinate
    xc = -1 + 2 * 5 / 7
    assert f[2 * 8 + 5, 2 + 4 * 3 + 1] == pytest.approx(math.sin(8 * xc), abs=1e-13)
    assert f[2 * 8 + 5, 4 + 4 * 3 + 0] == pytest.approx(math.cos(8 * (-1 + 2 * 2 / 7)), abs=1e-13)


def test_L0_reduces_to_a_relu_mlp_on_raw_coordinates_brute_force():
    M, dh, r = 3, 4, 2
    w_h, b_h, w_pq, w_pk = _weights(0, dh, r, 1)
    pq, pk, h, r_in = gen.forward(w_h, b_h, w_pq, w_pk, M, 0)
    for i in range(M * M):
        y, x = divmod(i, M)
        cy, cx = -1 + y, -1 + x                                    # linspace(-1, 1, 3) = -1, 0, 1
        hid = [max(0.0, cy * w_h[0][j] + cx * w_h[1][j] + b_h[j]) for j in range(dh)]
        for c in range(r):
            assert pq[i, c] == pytest.approx(sum(hid[j] * w_pq[j][c] for j in range(dh)), abs=1e-13)
            assert pk[i, c] == pytest.approx(sum(hid[j] * w_pk[j][c] for j in range(dh)), abs=1e-13)


def test_bias_has_rank_at_most_R_and_hidden_is_nonnegative():
    w = _weights(10, 32, 16, 2)
    pq, pk, h, _ = gen.forward(*w, 16, 10)
    assert (h >= 0).all() and np.linalg.matrix_rank(pq @ pk.T) <= 16    # "rank-factorized": the n x n bias has rank <= R


def test_forward_matches_library_linear_layers():
    L, dh, r, M = 10, 32, 16, 8
    w_h, b_h, w_pq, w_pk = _weights(L, dh, r, 3)
    pq, pk, _, r_in = gen.forward(w_h, b_h, w_pq, w_pk, M, L)
    t = torch.from_numpy(r_in)
    hid = torch.relu(torch.nn.functional.linear(t, torch.from_numpy(w_h).T, torch.from_numpy(b_h)))
    assert np.allclose(pq, torch.nn.functional.linear(hid, torch.from_numpy(w_pq).T).numpy(), atol=1e-12)
    assert np.allclose(pk, torch.nn.functional.linear(hid, torch.from_numpy(w_pk).T).numpy(), atol=1e-12)


def test_backward_matches_autograd_and_finite_differences():
    L, dh, r, M = 4, 8, 4, 5
    w = [torch.from_numpy(a).requires_grad_(True) for a in _weights(L, dh, r, 4)]
    rng = np.random.default_rng(5)
    dpq, dpk = rng.normal(size=(M * M, r)), rng.normal(size=(M * M, r))
    r_in = torch.from_numpy(gen.fourier_features(gen.coordinates(M), L))
    hid = torch.relu(r_in @ w[0] + w[1])
    loss = ((hid @ w[2]) * torch.from_numpy(dpq)).sum() + ((hid @ w[3]) * torch.from_numpy(dpk)).sum()
    loss.backward()
    got = gen.backward(*[a.detach().numpy() for a in w], dpq, dpk, M, L)
    for g, a in zip(got, w):
        assert np.allclose(g, a.grad.numpy(), atol=1e-11)
    # central finite differences on a few entries of every parameter
    base = [a.detach().numpy().copy() for a in w]
    def value(ws):
        pq, pk, _, _ = gen.forward(*ws, M, L)
        return (pq * dpq).sum() + (pk * dpk).sum()
    for k in range(4):
        flat_idx = [0, base[k].size // 2, base[k].size - 1]
        for fi in flat_idx:
            up, dn = [b.copy() for b in base], [b.copy() for b in base]
            up[k].reshape(-1)[fi] += 1e-6; dn[k].reshape(-1)[fi] -= 1e-6
            fd = (value(up) - value(dn)) / 2e-6
            assert got[k].reshape(-1)[fi] == pytest.approx(fd, rel=1e-5, abs=1e-7)


def test_planted_mistakes_are_caught():
    """A dropped cosine block, a pi in the frequencies or column-major tokens change the features."""
    x = gen.coordinates(4)
    good = gen.fourier_features(x, 3)
    with_pi = np.concatenate([x] + [fn((2.0 ** l) * np.pi * x) for l in range(3) for fn in (np.sin, np.cos)], axis=1)
    swapped = np.concatenate([x] + [fn((2.0 ** l) * x) for l in range(3) for fn in (np.cos, np.sin)], axis=1)
    assert not np.allclose(good, with_pi) and not np.allclose(good, swapped)
    col_major = gen.coordinates(4).reshape(4, 4, 2).transpose(1, 0, 2).reshape(-1, 2)
    assert not np.allclose(gen.coordinates(4), col_major)

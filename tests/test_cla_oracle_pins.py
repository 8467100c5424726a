"""Pins of the CLA gate oracle (oracle/cla_oracle.py, Eq. 8 / Eq. 9): library convolutions, closed forms, and
planted mistakes."""
import numpy as np
import pytest
import torch

from oracle import cla_oracle as cla


def rand_case(seed, B=2, H=5, W=7, D=8):
    rng = np.random.default_rng(seed)
    return (rng.standard_normal((B, H, W, D)), 0.4 * rng.standard_normal((D, 3, 3)), 0.2 * rng.standard_normal(D),
            0.3 * rng.standard_normal((D, D)), 0.2 * rng.standard_normal(D))


def torch_gate(x, w_dw, b_dw, w_pw, b_pw):
    D = x.shape[-1]
    t = torch.from_numpy(x).permute(0, 3, 1, 2)
    y = torch.nn.functional.conv2d(t, torch.from_numpy(w_dw)[:, None], torch.from_numpy(b_dw), padding=1, groups=D)
    z = torch.nn.functional.conv2d(y, torch.from_numpy(w_pw)[:, :, None, None], torch.from_numpy(b_pw))
    return torch.sigmoid(z).permute(0, 2, 3, 1).numpy()


@pytest.mark.parametrize("seed,shape", [(0, (2, 5, 7, 8)), (1, (1, 1, 1, 4)), (2, (1, 3, 1, 6)), (3, (1, 8, 16, 16))])
def test_gate_equals_library_convolutions(seed, shape):
    x, w_dw, b_dw, w_pw, b_pw = rand_case(seed, *shape)
    np.testing.assert_allclose(cla.gate(x, w_dw, b_dw, w_pw, b_pw), torch_gate(x, w_dw, b_dw, w_pw, b_pw), rtol=0, atol=1e-13)


def test_delta_filter_and_identity_matrix_give_sigmoid_of_x():
    x, _, _, _, _ = rand_case(4)
    D = x.shape[-1]
    w_dw = np.zeros((D, 3, 3)); w_dw[:, 1, 1] = 1.0
    g = cla.gate(x, w_dw, np.zeros(D), np.eye(D), np.zeros(D))
    np.testing.assert_allclose(g, 1 / (1 + np.exp(-x)), atol=1e-15)


def test_box_filter_on_constant_map_counts_neighbours():
    D = 3
    x = np.ones((1, 4, 5, D))
    y = cla.dwconv3x3(x, np.ones((D, 3, 3)), np.zeros(D))
    assert y[0, 0, 0, 0] == 4 and y[0, 0, 2, 1] == 6 and y[0, 2, 2, 2] == 9 and y[0, 3, 4, 0] == 4    # zero padding


def test_filter_orientation_is_cross_correlation():
    D = 2
    x = np.zeros((1, 3, 3, D)); x[0, 0, 2, :] = 1.0          # a single one at the top right
    w = np.zeros((D, 3, 3)); w[:, 0, 2] = 5.0                # the tap that looks up and to the right
    y = cla.dwconv3x3(x, w, np.zeros(D))
    assert y[0, 1, 1, 0] == 5.0 and np.count_nonzero(y[..., 0]) == 1


def test_pointwise_matrix_is_out_by_in():
    y = np.zeros((1, 1, 1, 3)); y[..., 1] = 2.0
    w = np.arange(9.0).reshape(3, 3)                          # w[out, in]
    np.testing.assert_allclose(cla.pwconv(y, w, np.zeros(3))[0, 0, 0], 2.0 * w[:, 1])


def test_gated_output_follows_the_channel_layout_of_the_heads():
    rng = np.random.default_rng(5)
    out = rng.standard_normal((1, 2, 2, 3, 4))
    g = rng.random((1, 2, 2, 12))
    got = cla.gated_output(out, g)
    assert got[0, 1, 0, 2, 3] == out[0, 1, 0, 2, 3] * g[0, 1, 0, 2 * 4 + 3]


def test_planted_mistakes_are_caught():
    x, w_dw, b_dw, w_pw, b_pw = rand_case(6)
    ref = torch_gate(x, w_dw, b_dw, w_pw, b_pw)
    wrong = [cla.gate(x, w_dw[:, ::-1, ::-1], b_dw, w_pw, b_pw),          # flipped filter (true convolution)
             cla.gate(x, w_dw, b_dw, w_pw.T, b_pw),                         # in/out swapped
             cla.gate(x, w_dw, np.zeros_like(b_dw), w_pw, b_pw),            # dropped bias
             cla.gate(x, w_dw.transpose(0, 2, 1), b_dw, w_pw, b_pw)]        # dy/dx swapped
    for w in wrong:
        assert np.abs(w - ref).max() > 1e-3

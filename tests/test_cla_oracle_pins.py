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


# ---- backward of Eq. 8 / Eq. 9: library autograd, finite differences, closed forms, planted mistakes ----

def torch_gate_bwd(x, w_dw, b_dw, w_pw, b_pw, dgate):
    D = x.shape[-1]
    ts = [torch.from_numpy(np.ascontiguousarray(a)).requires_grad_() for a in (x, w_dw, b_dw, w_pw, b_pw)]
    t = ts[0].permute(0, 3, 1, 2)
    y = torch.nn.functional.conv2d(t, ts[1][:, None], ts[2], padding=1, groups=D)
    z = torch.nn.functional.conv2d(y, ts[3][:, :, None, None], ts[4])
    g = torch.sigmoid(z).permute(0, 2, 3, 1)
    g.backward(torch.from_numpy(dgate))
    return [a.grad.numpy() for a in ts]


@pytest.mark.parametrize("seed,shape", [(10, (2, 5, 7, 8)), (11, (1, 1, 1, 4)), (12, (1, 1, 4, 6)), (13, (1, 8, 16, 16))])
def test_gate_bwd_equals_library_autograd(seed, shape):
    x, w_dw, b_dw, w_pw, b_pw = rand_case(seed, *shape)
    dgate = np.random.default_rng(seed + 100).standard_normal(x.shape)
    got = cla.gate_bwd(x, w_dw, b_dw, w_pw, b_pw, dgate)
    for a, b in zip(got, torch_gate_bwd(x, w_dw, b_dw, w_pw, b_pw, dgate)):
        np.testing.assert_allclose(a, b, rtol=0, atol=1e-12)


def test_gate_bwd_matches_central_differences_of_the_forward():
    args = list(rand_case(14, 1, 3, 4, 5))
    dgate = np.random.default_rng(15).standard_normal(args[0].shape)
    grads = cla.gate_bwd(*args, dgate)
    rng = np.random.default_rng(16)
    eps = 1e-6
    for which in range(5):
        for _ in range(6):
            idx = tuple(rng.integers(0, s) for s in args[which].shape)
            hi = [a.copy() for a in args]; hi[which][idx] += eps
            lo = [a.copy() for a in args]; lo[which][idx] -= eps
            fd = ((cla.gate(*hi) - cla.gate(*lo)) * dgate).sum() / (2 * eps)
            assert abs(fd - grads[which][idx]) < 1e-7


def test_gate_bwd_with_delta_filter_and_identity_matrix_is_the_sigmoid_slope():
    x, _, _, _, _ = rand_case(17)
    D = x.shape[-1]
    w_dw = np.zeros((D, 3, 3)); w_dw[:, 1, 1] = 1.0
    dgate = np.random.default_rng(18).standard_normal(x.shape)
    dx, dw_dw, db_dw, dw_pw, db_pw = cla.gate_bwd(x, w_dw, np.zeros(D), np.eye(D), np.zeros(D), dgate)
    s = 1 / (1 + np.exp(-x))
    dz = dgate * s * (1 - s)
    np.testing.assert_allclose(dx, dz, atol=1e-15)
    np.testing.assert_allclose(db_pw, dz.sum(axis=(0, 1, 2)), atol=1e-13)
    np.testing.assert_allclose(db_dw, db_pw, atol=1e-13)
    np.testing.assert_allclose(dw_pw, np.einsum("bhwo,bhwi->oi", dz, x), atol=1e-12)
    np.testing.assert_allclose(dw_dw[:, 1, 1], (dz * x).sum(axis=(0, 1, 2)), atol=1e-12)


def test_gate_bwd_single_pixel_gradient_spreads_over_the_filter_footprint():
    D = 2
    x = np.zeros((1, 5, 5, D))
    w_dw = np.arange(1.0, 19.0).reshape(D, 3, 3)
    dgate = np.zeros_like(x); dgate[0, 2, 3, :] = 4.0       # sigmoid'(0) = 1/4, identity matrix: dY = 1 at (2, 3)
    dx, *_ = cla.gate_bwd(x, w_dw, np.zeros(D), np.eye(D), np.zeros(D), dgate)
    # Y[2, 3] reads X[2 + ky - 1, 3 + kx - 1] through tap (ky, kx): the footprint is the filter itself, unflipped
    np.testing.assert_allclose(dx[0, 1:4, 2:5, 1], w_dw[1], atol=1e-15)
    assert np.count_nonzero(dx[..., 0]) == 9


def test_gated_output_bwd_is_the_product_rule():
    rng = np.random.default_rng(19)
    out = rng.standard_normal((1, 2, 3, 2, 4))
    g = rng.random((1, 2, 3, 8))
    dgo = rng.standard_normal(out.shape)
    dout, dg = cla.gated_output_bwd(out, g, dgo)
    assert dout[0, 1, 2, 1, 3] == dgo[0, 1, 2, 1, 3] * g[0, 1, 2, 7]
    assert dg[0, 1, 2, 7] == dgo[0, 1, 2, 1, 3] * out[0, 1, 2, 1, 3]
    eps = 1e-6
    o2 = out.copy(); o2[0, 0, 1, 1, 2] += eps
    fd = ((cla.gated_output(o2, g) - cla.gated_output(out, g)) * dgo).sum() / eps
    assert abs(fd - dout[0, 0, 1, 1, 2]) < 1e-8


def test_planted_mistakes_in_the_backward_are_caught():
    x, w_dw, b_dw, w_pw, b_pw = rand_case(20)
    dgate = np.random.default_rng(21).standard_normal(x.shape)
    ref = torch_gate_bwd(x, w_dw, b_dw, w_pw, b_pw, dgate)
    # the mistakes are planted in the inputs handed to the oracle: each must move at least one gradient
    wrong = [cla.gate_bwd(x, w_dw[:, ::-1, ::-1], b_dw, w_pw, b_pw, dgate),     # flipped filter
             cla.gate_bwd(x, w_dw, b_dw, w_pw.T, b_pw, dgate),                    # in/out swapped
             cla.gate_bwd(x, w_dw, b_dw, w_pw, b_pw, -dgate),                     # sign
             cla.gate_bwd(x, w_dw.transpose(0, 2, 1), b_dw, w_pw, b_pw, dgate)]   # dy/dx swapped
    for w in wrong:
        assert max(np.abs(a - b).max() for a, b in zip(w, ref)) > 1e-3

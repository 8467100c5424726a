"""GPU parity for Convolutional Local Attention (Eq. 8, Eq. 9): the gate kernel against the numpy oracle, and the
forward pass with the gate multiplied into its output against oracle attention times the same gate."""
import numpy as np
import pytest
import torch

from oracle import cla_oracle as cla
from paper_2603_06738_b200 import binding, synthetic
from paper_2603_06738_b200.synthetic import Workload

from parity_util import compare, make, oracle_fwd, to_f64, widths_fit_tensor_cores

pytestmark = pytest.mark.gpu


def gate_inputs(seed, B, H, W, D):
    x = synthetic.bf16_tensor(seed, "x", (B, H, W, D), 1.0)
    rng = np.random.default_rng(seed)
    w_dw = np.float32(rng.normal(0, 0.35, (D, 3, 3)))
    b_dw = np.float32(rng.normal(0, 0.2, D))
    w_pw = np.float32(rng.normal(0, 1.5 / np.sqrt(D), (D, D)))
    b_pw = np.float32(rng.normal(0, 0.3, D))
    return x, [w_dw, b_dw, w_pw, b_pw]


# the last three shapes give every persistent CTA several tiles (the benchmark shape: 576 tiles on 148 CTAs)
@pytest.mark.parametrize("B,H,W,D", [(1, 8, 16, 64), (2, 16, 32, 192), (1, 24, 48, 128), (3, 40, 16, 192), (1, 96, 96, 192),
                                     (8, 96, 96, 192), (2, 160, 160, 64), (4, 88, 96, 128),
                                     (2, 16, 32, 180), (1, 24, 48, 96), (1, 8, 16, 30)])      # 6 x 30, 6 x 16 channels: zero-padded copies
def test_gate_matches_the_oracle(B, H, W, D):
    x, ws = gate_inputs(200 + D + H, B, H, W, D)
    g = binding.rib_cla_gate(x.cuda(), *[torch.from_numpy(w).cuda() for w in ws])
    torch.cuda.synchronize()
    assert binding.rib_query_status() == 0
    ref = cla.gate(to_f64(x), *ws)
    # bf16 operands of the point-wise matrix and a bf16 result in (0, 1)
    compare("gate", to_f64(g), ref, max_abs=1e-2, rel_l2=5e-3)
    assert float(g.float().min()) >= 0.0 and float(g.float().max()) <= 1.0


def test_gate_border_pixels_see_zero_padding():
    """A map of ones with a box filter: the depth-wise sum is 4, 6 or 9 depending on the border, and an identity
    point-wise matrix passes it on, so the gate is sigmoid of those counts."""
    B, H, W, D = 1, 8, 16, 64
    x = torch.ones((B, H, W, D), dtype=torch.bfloat16, device="cuda")
    w_dw = torch.full((D, 3, 3), 0.25, device="cuda")
    g = binding.rib_cla_gate(x, w_dw, torch.zeros(D, device="cuda"), torch.eye(D, device="cuda"), torch.zeros(D, device="cuda"))
    torch.cuda.synchronize()
    sig = lambda z: 1 / (1 + np.exp(-z))
    got = to_f64(g)
    assert abs(got[0, 0, 0, 5] - sig(1.0)) < 4e-3 and abs(got[0, 0, 7, 9] - sig(1.5)) < 4e-3
    assert abs(got[0, 3, 8, 63] - sig(2.25)) < 4e-3 and abs(got[0, 7, 15, 0] - sig(1.0)) < 4e-3


@pytest.mark.parametrize("path", ["auto", "generic"])
@pytest.mark.parametrize("wl", [Workload("gated_w16_s8", 2, 32, 48, 2, 32, 16, 16, 8, seed=210),
                                Workload("gated_w32_rank32", 1, 64, 32, 6, 32, 32, 32, 16, seed=211),
                                Workload("gated_w8_generic", 1, 16, 24, 3, 16, 8, 8, 3, seed=212),
                                Workload("gated_w16_headwise", 1, 32, 32, 3, 32, 16, 16, 0, seed=215, headwise=True),
                                Workload("gated_w16_d16_r24", 1, 32, 32, 4, 16, 24, 16, 8, seed=216),
                                Workload("gated_w16_d30_r18", 1, 32, 32, 6, 30, 18, 16, 8, seed=217)], ids=lambda w: w.name)
def test_gated_forward_is_attention_times_the_gate(wl, path):
    cpu, gpu = make(wl, with_dout=False)
    D = wl.heads * wl.d
    gate = synthetic.bf16_tensor(wl.seed, "gate", (wl.B, wl.H, wl.W, D), 0.3).abs().clamp(max=1.0).to(torch.bfloat16)
    binding.rib_set_path(binding.RIB_PATH_GENERIC if path == "generic" else binding.RIB_PATH_NONE)
    try:
        out, lse = binding.rib_window_attn_fwd_gated(gpu["q"], gpu["k"], gpu["v"], gpu["pq"], gpu["pk"], gate.cuda(), wl.window, wl.shift)
        used = binding.rib_last_path()
    finally:
        binding.rib_set_path(binding.RIB_PATH_NONE)
    torch.cuda.synchronize()
    assert binding.rib_query_status() == 0
    fast = path == "auto" and widths_fit_tensor_cores(wl.d, wl.r) and wl.window % 16 == 0 and wl.shift % 8 == 0
    assert used == (binding.RIB_PATH_SM100 if fast else binding.RIB_PATH_GENERIC)
    ref_out, ref_lse = oracle_fwd(cpu, wl)
    compare("out", to_f64(out), cla.gated_output(ref_out, to_f64(gate)))
    compare("lse", to_f64(lse), ref_lse)


def test_gate_then_gated_forward_end_to_end():
    """Eq. 8 and Eq. 9 chained on the GPU: features -> gate -> gated attention output, against the oracles chained."""
    wl = Workload("cla_chain", 1, 32, 32, 6, 32, 16, 16, 8, seed=213)
    cpu, gpu = make(wl, with_dout=False)
    x, ws = gate_inputs(214, wl.B, wl.H, wl.W, wl.heads * wl.d)
    g = binding.rib_cla_gate(x.cuda(), *[torch.from_numpy(w).cuda() for w in ws])
    out, _ = binding.rib_window_attn_fwd_gated(gpu["q"], gpu["k"], gpu["v"], gpu["pq"], gpu["pk"], g, wl.window, wl.shift)
    torch.cuda.synchronize()
    assert binding.rib_query_status() == 0
    ref = cla.gated_output(oracle_fwd(cpu, wl)[0], cla.gate(to_f64(x), *ws))
    compare("gated out", to_f64(out), ref)


def test_gate_rejects_unsupported_sizes():
    lib = binding.library()
    x = torch.zeros(1 << 16, dtype=torch.bfloat16, device="cuda")
    w = torch.zeros(1 << 16, dtype=torch.float32, device="cuda")
    ptrs = [x.data_ptr()] + [w.data_ptr()] * 4
    launches = binding.rib_kernel_launches()
    assert lib.rib_cla_gate(*ptrs, 1, 8, 16, 95, x.data_ptr(), None) == -3     # an odd number of channels
    assert lib.rib_cla_gate(*ptrs, 1, 8, 16, 200, x.data_ptr(), None) == -3    # more than 192 channels
    assert lib.rib_cla_gate(*ptrs, 1, 8, 24, 64, x.data_ptr(), None) == -3     # W not a multiple of 16
    assert lib.rib_cla_gate(*ptrs, 1, 12, 16, 64, x.data_ptr(), None) == -3    # H not a multiple of 8
    assert lib.rib_cla_gate(*ptrs, 0, 8, 16, 64, x.data_ptr(), None) == -2
    assert lib.rib_cla_gate(None, *ptrs[1:], 1, 8, 16, 64, x.data_ptr(), None) == -1
    assert binding.rib_kernel_launches() == launches


# ---- backward of Eq. 8 and Eq. 9 ----

def dgate_input(seed, shape):
    return synthetic.bf16_tensor(seed, "gate", shape, 1.0)


@pytest.mark.parametrize("path", ["auto", "generic"])
@pytest.mark.parametrize("B,H,W,D", [(1, 5, 7, 64), (2, 16, 32, 192), (1, 24, 47, 128), (3, 9, 16, 192), (1, 1, 1, 64),
                                     (1, 96, 96, 192), (2, 40, 56, 64),
                                     # several tiles per persistent CTA / block, the last one with ragged H and W
                                     (8, 96, 96, 192), (2, 160, 160, 64), (4, 90, 100, 128),
                                     (2, 19, 32, 180), (1, 24, 48, 96)])         # 6 x 30, 6 x 16 channels: zero-padded copies
def test_gate_backward_matches_the_oracle(B, H, W, D, path):
    x, ws = gate_inputs(300 + D + H, B, H, W, D)
    dgate = dgate_input(301 + D + H, (B, H, W, D))
    binding.rib_set_path(binding.RIB_PATH_GENERIC if path == "generic" else binding.RIB_PATH_NONE)
    try:
        got = binding.rib_cla_gate_bwd(x.cuda(), *[torch.from_numpy(w).cuda() for w in ws], dgate.cuda())
        used = binding.rib_last_path()
    finally:
        binding.rib_set_path(binding.RIB_PATH_NONE)
    torch.cuda.synchronize()
    assert binding.rib_query_status() == 0
    assert used == (binding.RIB_PATH_GENERIC if path == "generic" else binding.RIB_PATH_SM100)
    ref = cla.gate_bwd(to_f64(x), *ws, to_f64(dgate))
    compare("dx", to_f64(got[0]), ref[0], max_abs=1e-2 * max(1.0, np.abs(ref[0]).max()))
    for name, g, r in zip(("dw_dw", "db_dw", "dw_pw", "db_pw"), got[1:], ref[1:]):
        if path == "generic":
            # fp32 products and fp32 sums over the pixels, against float64
            compare(name, to_f64(g), r, max_abs=1e-3 * max(1.0, np.abs(r).max()), rel_l2=1e-4)
        else:
            # Y, dZ and the point-wise matrix enter the MMAs as bf16 (fp32 accumulation): the bar of the attention outputs
            compare(name, to_f64(g), r, max_abs=1e-2 * max(1.0, np.abs(r).max()), rel_l2=5e-3)


def test_gate_backward_overwrites_its_outputs_and_repeats():
    B, H, W, D = 1, 16, 16, 64
    x, ws = gate_inputs(310, B, H, W, D)
    dgate = dgate_input(311, (B, H, W, D))
    args = [x.cuda(), *[torch.from_numpy(w).cuda() for w in ws], dgate.cuda()]
    first = [t.clone() for t in binding.rib_cla_gate_bwd(*args)]
    second = binding.rib_cla_gate_bwd(*args)
    torch.cuda.synchronize()
    assert torch.equal(first[0], second[0])                                       # dx has a fixed summation order
    for a, b in zip(first[1:], second[1:]):                                       # atomics: equal up to rounding
        assert torch.allclose(a, b, rtol=1e-4, atol=1e-5)


@pytest.mark.parametrize("shape", [(1, 8, 16, 2, 32), (2, 5, 7, 6, 32), (1, 96, 96, 6, 32)])
def test_product_and_its_backward_match_the_oracle(shape):
    B, H, W, heads, d = shape
    out = synthetic.bf16_tensor(320, "x", shape, 1.0)
    gate = synthetic.bf16_tensor(321, "gate", (B, H, W, heads * d), 0.3).abs().clamp(max=1.0).to(torch.bfloat16)
    dgo = synthetic.bf16_tensor(322, "dout", shape, 1.0)
    prod = binding.rib_cla_product(out.cuda(), gate.cuda())
    dout, dgate = binding.rib_cla_product_bwd(out.cuda(), gate.cuda(), dgo.cuda())
    torch.cuda.synchronize()
    ref_dout, ref_dgate = cla.gated_output_bwd(to_f64(out), to_f64(gate), to_f64(dgo))
    # one bf16 rounding of an exact fp32 product: the GPU result is the correctly rounded oracle value
    for got, ref in ((prod, cla.gated_output(to_f64(out), to_f64(gate))), (dout, ref_dout), (dgate, ref_dgate)):
        want = torch.from_numpy(ref).to(torch.bfloat16)
        assert torch.equal(got.cpu().reshape(want.shape), want)


def test_gate_backward_rejects_unsupported_channels_without_launching():
    lib = binding.library()
    x = torch.zeros(1 << 16, dtype=torch.bfloat16, device="cuda")
    w = torch.zeros(1 << 16, dtype=torch.float32, device="cuda")
    launches = binding.rib_kernel_launches()
    assert lib.rib_cla_gate_bwd(x.data_ptr(), *[w.data_ptr()] * 4, x.data_ptr(), 1, 4, 4, 95, x.data_ptr(), *[w.data_ptr()] * 4,
                                w.data_ptr(), 1 << 18, None) == -3
    assert binding.rib_kernel_launches() == launches


def test_training_chain_matches_the_oracles_chained():
    """Features -> gate, attention -> out, out o gate, and the whole way back on the GPU, against the oracles chained in
    float64 (no intermediate rounded to bf16 on the oracle's side)."""
    from oracle import rib_oracle as orc
    wl = Workload("cla_train_chain", 2, 32, 48, 2, 32, 16, 16, 8, seed=330)
    cpu, gpu = make(wl)
    D = wl.heads * wl.d
    x, ws = gate_inputs(331, wl.B, wl.H, wl.W, D)
    wg = [torch.from_numpy(w).cuda() for w in ws]
    gate = binding.rib_cla_gate(x.cuda(), *wg)
    out, lse = binding.rib_window_attn_fwd(gpu["q"], gpu["k"], gpu["v"], gpu["pq"], gpu["pk"], wl.window, wl.shift)
    out_gated = binding.rib_cla_product(out, gate)
    dout_attn, dgate = binding.rib_cla_product_bwd(out, gate, gpu["dout"])            # dout: the gradient of out_gated
    grads_gate = binding.rib_cla_gate_bwd(x.cuda(), *wg, dgate)
    grads_attn = binding.rib_window_attn_bwd(gpu["q"], gpu["k"], gpu["v"], gpu["pq"], gpu["pk"], out, lse, dout_attn, wl.window, wl.shift)
    torch.cuda.synchronize()
    assert binding.rib_query_status() == 0

    ref_out, _ = oracle_fwd(cpu, wl)
    ref_gate = cla.gate(to_f64(x), *ws)
    compare("gated out", to_f64(out_gated), cla.gated_output(ref_out, ref_gate))
    ref_dout, ref_dgate = cla.gated_output_bwd(ref_out, ref_gate, to_f64(cpu["dout"]))
    ref_gate_grads = cla.gate_bwd(to_f64(x), *ws, ref_dgate)
    ref_attn_grads = orc.bwd(*(to_f64(cpu[k]) for k in ("q", "k", "v", "pq", "pk")), ref_dout, wl.window, wl.shift)
    for name, g, r in zip(("dx", "dw_dw", "db_dw", "dw_pw", "db_pw"), grads_gate, ref_gate_grads):
        compare(name, to_f64(g), r, max_abs=1e-2 * max(1.0, np.abs(r).max()))
    for name, g, r in zip(("dq", "dk", "dv", "dpq", "dpk"), grads_attn, ref_attn_grads):
        compare(name, to_f64(g), r, max_abs=1e-2 * max(1.0, np.abs(r).max()))


def test_gate_backward_with_a_workspace_that_is_only_16_byte_aligned():
    """The workspace is promised 16-byte alignment only; the kernel's 32-byte stores must then not be used."""
    B, H, W, D = 1, 16, 24, 192
    x, ws = gate_inputs(340, B, H, W, D)
    dgate = dgate_input(341, (B, H, W, D))
    args = [x.cuda(), *[torch.from_numpy(w).cuda() for w in ws], dgate.cuda()]
    need = binding.library().rib_cla_gate_bwd_workspace(B, H, W, D)
    buf = torch.empty(need + 64, dtype=torch.uint8, device="cuda")
    off = 16 if buf.data_ptr() % 32 == 0 else 0
    assert (buf.data_ptr() + off) % 32 == 16
    plain = [t.clone() for t in binding.rib_cla_gate_bwd(*args)]
    shifted = binding.rib_cla_gate_bwd(*args, workspace=buf[off:])
    torch.cuda.synchronize()
    assert binding.rib_query_status() == 0
    assert torch.equal(plain[0], shifted[0])
    for a, b in zip(plain[1:], shifted[1:]):
        assert torch.allclose(a, b, rtol=1e-4, atol=1e-5)

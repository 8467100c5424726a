"""GPU parity for Convolutional Local Attention (Eq. 8, Eq. 9): the gate kernel against the numpy oracle, and the
forward pass with the gate multiplied into its output against oracle attention times the same gate."""
import numpy as np
import pytest
import torch

from oracle import cla_oracle as cla
from paper_2603_06738_b200 import binding, synthetic
from paper_2603_06738_b200.synthetic import Workload

from parity_util import compare, make, oracle_fwd, to_f64

pytestmark = pytest.mark.gpu


def gate_inputs(seed, B, H, W, D):
    x = synthetic.bf16_tensor(seed, "x", (B, H, W, D), 1.0)
    rng = np.random.default_rng(seed)
    w_dw = np.float32(rng.normal(0, 0.35, (D, 3, 3)))
    b_dw = np.float32(rng.normal(0, 0.2, D))
    w_pw = np.float32(rng.normal(0, 1.5 / np.sqrt(D), (D, D)))
    b_pw = np.float32(rng.normal(0, 0.3, D))
    return x, [w_dw, b_dw, w_pw, b_pw]


@pytest.mark.parametrize("B,H,W,D", [(1, 8, 16, 64), (2, 16, 32, 192), (1, 24, 48, 128), (3, 40, 16, 192), (1, 96, 96, 192)])
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
                                Workload("gated_w16_headwise", 1, 32, 32, 3, 32, 16, 16, 0, seed=215, headwise=True)], ids=lambda w: w.name)
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
    fast = path == "auto" and wl.d == 32 and wl.window % 16 == 0 and wl.shift % 8 == 0
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
    assert lib.rib_cla_gate(*ptrs, 1, 8, 16, 96, x.data_ptr(), None) == -3     # channels not 64, 128 or 192
    assert lib.rib_cla_gate(*ptrs, 1, 8, 24, 64, x.data_ptr(), None) == -3     # W not a multiple of 16
    assert lib.rib_cla_gate(*ptrs, 1, 12, 16, 64, x.data_ptr(), None) == -3    # H not a multiple of 8
    assert lib.rib_cla_gate(*ptrs, 0, 8, 16, 64, x.data_ptr(), None) == -2
    assert lib.rib_cla_gate(None, *ptrs[1:], 1, 8, 16, 64, x.data_ptr(), None) == -1
    assert binding.rib_kernel_launches() == launches

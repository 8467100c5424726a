"""GPU parity for feature maps whose sides are not multiples of the window: rib_window_attn_fwd_padded against the
numpy oracle of the same reading (positions of the extended map beyond the image are not tokens), on the tcgen05
kernel (H, W multiples of 8) and on the any-shape kernel, every element."""
import numpy as np
import pytest
import torch

from oracle import rib_padded_oracle as pad
from paper_2603_06738_b200 import binding, synthetic
from paper_2603_06738_b200.synthetic import Workload

from parity_util import compare, to_f64, widths_fit_tensor_cores

pytestmark = pytest.mark.gpu

# name, B, H, W, heads, d, r, window, shift
CASES = [
    Workload("p_6x10_w4", 2, 6, 10, 2, 16, 8, 4, 0, seed=61),
    Workload("p_7x5_w4_s1", 1, 7, 5, 1, 8, 8, 4, 1, seed=62),
    Workload("p_20x28_w8_s3", 1, 20, 28, 3, 32, 16, 8, 3, seed=63),
    Workload("p_3x3_w4", 1, 3, 3, 2, 8, 8, 4, 0, seed=64),                       # one window, 9 of 16 positions real
    Workload("p_40x56_w16", 2, 40, 56, 2, 32, 16, 16, 0, seed=65),               # tcgen05 shapes from here on
    Workload("p_40x56_w16_s8", 1, 40, 56, 3, 32, 16, 16, 8, seed=66),
    Workload("p_72x88_w32_s16", 1, 72, 88, 3, 32, 16, 32, 16, seed=67),
    Workload("p_56x104_w48_s24_r32", 1, 56, 104, 2, 32, 32, 48, 24, seed=68),
    Workload("p_40x24_w32_headwise", 1, 40, 24, 3, 32, 16, 32, 0, seed=69, headwise=True),
    Workload("p_8x8_w16", 1, 8, 8, 1, 32, 16, 16, 0, seed=70),                    # a quarter of one window
    Workload("p_120x200_w64", 1, 120, 200, 2, 32, 16, 64, 0, seed=71),            # 16:9-like frame, 64 x 64 windows
    Workload("p_8x24_w16", 2, 8, 24, 2, 32, 16, 16, 0, seed=73),                  # every item has one key block with tokens
    Workload("p_8x24_w16_s8", 2, 8, 24, 2, 32, 16, 16, 8, seed=74),
    Workload("p_88x40_w32_s8", 2, 88, 40, 2, 32, 16, 32, 8, seed=75),             # whole query tiles in the extension
    Workload("p_40x56_w16_d16_r24", 1, 40, 56, 3, 16, 24, 16, 8, seed=77),         # narrow head, rank 24
    Workload("p_40x56_w16_d30_r34", 1, 40, 56, 3, 30, 34, 16, 8, seed=78),         # 60-byte rows: zero-padded copies, rank tail in the spare channels
]


@pytest.mark.parametrize("wl", CASES, ids=lambda w: w.name)
@pytest.mark.parametrize("path", ["auto", "generic"])
def test_padded_forward_every_element(wl, path):
    cpu = synthetic.make_inputs(wl, with_dout=False)
    gpu = {k: v.cuda() for k, v in cpu.items()}
    binding.rib_set_path(binding.RIB_PATH_GENERIC if path == "generic" else binding.RIB_PATH_NONE)
    try:
        out, lse = binding.rib_window_attn_fwd_padded(gpu["q"], gpu["k"], gpu["v"], gpu["pq"], gpu["pk"], wl.window, wl.shift)
        used = binding.rib_last_path()
    finally:
        binding.rib_set_path(binding.RIB_PATH_NONE)
    torch.cuda.synchronize()
    assert binding.rib_query_status() == 0
    fast = (path == "auto" and widths_fit_tensor_cores(wl.d, wl.r) and wl.window % 16 == 0
            and wl.shift % 8 == 0 and wl.H % 8 == 0 and wl.W % 8 == 0)
    assert used == (binding.RIB_PATH_SM100 if fast else binding.RIB_PATH_GENERIC)
    ref_out, ref_lse = pad.fwd(*(to_f64(cpu[k]) for k in ("q", "k", "v", "pq", "pk")), wl.window, wl.shift)
    assert np.isfinite(ref_out).all() and np.isfinite(ref_lse).all()      # every real token belongs to one window
    compare("out", to_f64(out), ref_out)
    compare("lse", to_f64(lse), ref_lse)


BWD_CASES = [wl for wl in CASES if wl.H * wl.W <= 72 * 88]


@pytest.mark.parametrize("wl", BWD_CASES, ids=lambda w: w.name)
@pytest.mark.parametrize("path", ["auto", "generic"])
def test_padded_backward_every_element(wl, path):
    """Backward on maps that are not multiples of the window, against the numpy oracle, on both kernel families."""
    cpu = synthetic.make_inputs(wl, with_dout=True)
    gpu = {k: v.cuda() for k, v in cpu.items()}
    out, lse = binding.rib_window_attn_fwd_padded(gpu["q"], gpu["k"], gpu["v"], gpu["pq"], gpu["pk"], wl.window, wl.shift)
    binding.rib_set_path(binding.RIB_PATH_GENERIC if path == "generic" else binding.RIB_PATH_NONE)
    try:
        dq, dk, dv, dpq, dpk = binding.rib_window_attn_bwd_padded(gpu["q"], gpu["k"], gpu["v"], gpu["pq"], gpu["pk"], out, lse,
                                                                  gpu["dout"], wl.window, wl.shift)
        used = binding.rib_last_path()
    finally:
        binding.rib_set_path(binding.RIB_PATH_NONE)
    torch.cuda.synchronize()
    assert binding.rib_query_status() == 0
    fast = (path == "auto" and widths_fit_tensor_cores(wl.d, wl.r) and wl.window % 16 == 0
            and wl.shift % 8 == 0 and wl.H % 8 == 0 and wl.W % 8 == 0)
    assert used == (binding.RIB_PATH_SM100 if fast else binding.RIB_PATH_GENERIC)
    ref = pad.bwd(*(to_f64(cpu[k]) for k in ("q", "k", "v", "pq", "pk", "dout")), wl.window, wl.shift)
    assert all(np.isfinite(r).all() for r in ref)
    for name, got, want in zip(("dq", "dk", "dv"), (dq, dk, dv), ref[:3]):
        compare(name, to_f64(got), want)
    scale = max(1.0, float(np.abs(ref[3]).max()), float(np.abs(ref[4]).max()))
    compare("dpq", to_f64(dpq), ref[3], max_abs=1e-2 * scale)
    compare("dpk", to_f64(dpk), ref[4], max_abs=1e-2 * scale)


def test_padded_backward_entry_point_on_a_divisible_map_is_the_plain_call():
    wl = Workload("p_bwd_divisible", 1, 64, 32, 3, 32, 16, 32, 8, seed=76)
    gpu = {k: v.cuda() for k, v in synthetic.make_inputs(wl, with_dout=True).items()}
    out, lse = binding.rib_window_attn_fwd(gpu["q"], gpu["k"], gpu["v"], gpu["pq"], gpu["pk"], wl.window, wl.shift)
    a = binding.rib_window_attn_bwd(gpu["q"], gpu["k"], gpu["v"], gpu["pq"], gpu["pk"], out, lse, gpu["dout"], wl.window, wl.shift)
    b = binding.rib_window_attn_bwd_padded(gpu["q"], gpu["k"], gpu["v"], gpu["pq"], gpu["pk"], out, lse, gpu["dout"], wl.window, wl.shift)
    torch.cuda.synchronize()
    assert binding.rib_last_path() == binding.RIB_PATH_SM100
    assert torch.equal(a[1], b[1]) and torch.equal(a[2], b[2])     # dk, dv: bit-reproducible
    compare("dq", to_f64(b[0]), to_f64(a[0]), max_abs=4e-3, rel_l2=1e-3)


def test_divisible_map_through_the_padded_entry_point_is_the_plain_call():
    wl = Workload("p_divisible", 2, 64, 32, 3, 32, 16, 32, 8, seed=72)
    gpu = {k: v.cuda() for k, v in synthetic.make_inputs(wl, with_dout=False).items()}
    a = binding.rib_window_attn_fwd(gpu["q"], gpu["k"], gpu["v"], gpu["pq"], gpu["pk"], wl.window, wl.shift)
    b = binding.rib_window_attn_fwd_padded(gpu["q"], gpu["k"], gpu["v"], gpu["pq"], gpu["pk"], wl.window, wl.shift)
    torch.cuda.synchronize()
    assert binding.rib_last_path() == binding.RIB_PATH_SM100
    assert torch.equal(a[0], b[0]) and torch.equal(a[1], b[1])


def test_plain_entry_points_still_reject_partial_windows():
    x = torch.zeros(40 * 56 * 32, dtype=torch.bfloat16, device="cuda")
    pos = torch.zeros(256 * 16, dtype=torch.bfloat16, device="cuda")
    lib = binding.library()
    rc = lib.rib_window_attn_fwd(x.data_ptr(), x.data_ptr(), x.data_ptr(), pos.data_ptr(), pos.data_ptr(),
                                 1, 40, 56, 1, 32, 16, 16, 0, x.data_ptr(), None, None)
    assert rc == -2      # RIB_ERR_SHAPE
    assert lib.rib_window_attn_bwd_workspace(1, 40, 56, 1, 32, 16, 16) == 0


def test_window_cycle_driver_runs_the_six_layers_of_a_block():
    """Sec. 3.3: the window size cycles over the layers of a block.  One call enqueues all six layers (and one more call their
    backward passes); every layer is
    compared with the oracle (64 does not divide the 96-row map: that layer runs on partial windows), and a repeated
    call encodes no tensor map."""
    B, H, W, heads, d, r = 1, 96, 64, 2, 32, 16
    windows = [16, 32, 64, 16, 32, 64]
    layers = []
    for l, win in enumerate(windows):
        wl = Workload(f"cycle_l{l}", B, H, W, heads, d, r, win, 0, seed=300 + l)
        cpu = synthetic.make_inputs(Workload(wl.name, B, win, win, heads, d, r, win, 0, seed=300 + l), False)   # tables of n = win^2 rows
        img = synthetic.make_inputs(Workload(wl.name, B, 96, 96, heads, d, r, 96, 0, seed=310 + l), False)
        layers.append({"q": img["q"][:, :H, :W].contiguous(), "k": img["k"][:, :H, :W].contiguous(), "v": img["v"][:, :H, :W].contiguous(),
                       "pq": cpu["pq"], "pk": cpu["pk"]})
    dev = [{k: v.cuda() for k, v in layer.items()} for layer in layers]
    args = [[layer[k] for layer in dev] for k in ("q", "k", "v", "pq", "pk")]
    launches = binding.rib_kernel_launches()
    outs, lses = binding.rib_window_cycle_fwd(*args, windows)
    torch.cuda.synchronize()
    assert binding.rib_query_status() == 0 and binding.rib_kernel_launches() == launches + 6
    for l, win in enumerate(windows):
        f64 = {k: to_f64(v) for k, v in layers[l].items()}
        ref_out, ref_lse = pad.fwd(f64["q"], f64["k"], f64["v"], f64["pq"], f64["pk"], win, 0)
        compare(f"layer {l} (window {win}) out", to_f64(outs[l]), ref_out)
        compare(f"layer {l} (window {win}) lse", to_f64(lses[l]), ref_lse)
    _, misses = binding.rib_tensor_map_cache_counts()
    binding.rib_window_cycle_fwd(*args, windows)
    torch.cuda.synchronize()
    assert binding.rib_tensor_map_cache_counts()[1] == misses      # q, k, v and Pk of every layer were mapped by the first call
    # the backward passes of the same six layers in one call, sharing one workspace
    douts = [synthetic.bf16_tensor(320 + l, "dout", (B, H, W, heads, d), 1.0) for l in range(len(windows))]
    launches = binding.rib_kernel_launches()
    grads = binding.rib_window_cycle_bwd(*args, outs, lses, [t.cuda() for t in douts], windows)
    torch.cuda.synchronize()
    assert binding.rib_query_status() == 0 and binding.rib_kernel_launches() == launches + 18
    for l, win in enumerate(windows):
        f64 = {k: to_f64(v) for k, v in layers[l].items()}
        ref = pad.bwd(f64["q"], f64["k"], f64["v"], f64["pq"], f64["pk"], to_f64(douts[l]), win, 0)
        for name, got, want in zip(("dq", "dk", "dv"), (grads[0][l], grads[1][l], grads[2][l]), ref[:3]):
            compare(f"layer {l} (window {win}) {name}", to_f64(got), want)
        scale = max(1.0, float(np.abs(ref[3]).max()), float(np.abs(ref[4]).max()))
        compare(f"layer {l} (window {win}) dpq", to_f64(grads[3][l]), ref[3], max_abs=1e-2 * scale)
        compare(f"layer {l} (window {win}) dpk", to_f64(grads[4][l]), ref[4], max_abs=1e-2 * scale)

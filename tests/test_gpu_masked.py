"""GPU parity for shifted windows whose wrapped parts do not attend to each other: rib_window_attn_fwd_masked and
rib_window_attn_bwd_masked against the numpy oracle of that reading, every element, on the tcgen05 kernels
(shift a multiple of 8) and on the any-shape kernels (any shift)."""
import numpy as np
import pytest
import torch

from oracle import rib_masked_oracle as msk
from oracle import rib_oracle as orc
from paper_2603_06738_b200 import binding, synthetic
from paper_2603_06738_b200.synthetic import Workload

from parity_util import compare, to_f64, widths_fit_tensor_cores

pytestmark = pytest.mark.gpu

# name, B, H, W, heads, d, r, window, shift
CASES = [
    Workload("m_8x12_w4_s1", 2, 8, 12, 2, 16, 8, 4, 1, seed=81),
    Workload("m_16x16_w8_s3", 1, 16, 16, 3, 32, 16, 8, 3, seed=82),
    Workload("m_8x8_w8_s4", 1, 8, 8, 1, 8, 8, 8, 4, seed=83),                    # one window holding all four parts
    Workload("m_32x48_w16_s8", 2, 32, 48, 2, 32, 16, 16, 8, seed=84),            # tcgen05 shapes from here on
    Workload("m_64x64_w32_s16", 1, 64, 64, 3, 32, 16, 32, 16, seed=85),
    Workload("m_64x96_w32_s8", 1, 64, 96, 2, 32, 16, 32, 8, seed=86),
    Workload("m_64x32_w32_s24", 2, 64, 32, 2, 32, 16, 32, 24, seed=87),          # one window column: every window wraps in x
    Workload("m_96x48_w48_s24_r32", 1, 96, 48, 2, 32, 32, 48, 24, seed=88),
    Workload("m_64x64_w32_s16_headwise", 1, 64, 64, 3, 32, 16, 32, 16, seed=89, headwise=True),
    Workload("m_128x64_w64_s32", 1, 128, 64, 2, 32, 16, 64, 32, seed=90),
    Workload("m_64x64_w32_s0", 1, 64, 64, 2, 32, 16, 32, 0, seed=91),            # no shift: nothing is masked
    Workload("m_64x32_w32_s16_d16_r24", 1, 64, 32, 3, 16, 24, 32, 16, seed=93),  # narrow head, rank 24
    Workload("m_64x32_w32_s16_d30_r18", 1, 64, 32, 3, 30, 18, 32, 16, seed=94),  # 60-byte rows: zero-padded copies
]


def is_fast(wl, path):
    return path != "generic" and widths_fit_tensor_cores(wl.d, wl.r) and wl.window % 16 == 0 and wl.shift % 8 == 0


@pytest.mark.parametrize("wl", CASES, ids=lambda w: w.name)
@pytest.mark.parametrize("path", ["auto", "exact", "generic"])
def test_masked_forward_every_element(wl, path):
    if path == "exact" and not is_fast(wl, path):
        pytest.skip("the exact softmax form is a form of the tcgen05 kernel")
    cpu = synthetic.make_inputs(wl, with_dout=False)
    gpu = {k: v.cuda() for k, v in cpu.items()}
    binding.rib_set_path({"auto": binding.RIB_PATH_NONE, "exact": binding.RIB_PATH_SM100_EXACT, "generic": binding.RIB_PATH_GENERIC}[path])
    try:
        out, lse = binding.rib_window_attn_fwd_masked(gpu["q"], gpu["k"], gpu["v"], gpu["pq"], gpu["pk"], wl.window, wl.shift)
        used = binding.rib_last_path()
    finally:
        binding.rib_set_path(binding.RIB_PATH_NONE)
    torch.cuda.synchronize()
    assert binding.rib_query_status() == 0
    assert used == (binding.RIB_PATH_SM100 if is_fast(wl, path) else binding.RIB_PATH_GENERIC)
    ref_out, ref_lse = msk.fwd(*(to_f64(cpu[k]) for k in ("q", "k", "v", "pq", "pk")), wl.window, wl.shift)
    compare("out", to_f64(out), ref_out)
    compare("lse", to_f64(lse), ref_lse)
    if wl.shift:
        # the mask matters on this input: the unmasked oracle differs by far more than the tolerance
        plain, _ = orc.fwd(*(to_f64(cpu[k]) for k in ("q", "k", "v", "pq", "pk")), wl.window, wl.shift)
        assert np.abs(plain - ref_out).max() > 5e-2


@pytest.mark.parametrize("wl", CASES, ids=lambda w: w.name)
@pytest.mark.parametrize("path", ["auto", "generic"])
def test_masked_backward_every_element(wl, path):
    cpu = synthetic.make_inputs(wl, with_dout=True)
    gpu = {k: v.cuda() for k, v in cpu.items()}
    out, lse = binding.rib_window_attn_fwd_masked(gpu["q"], gpu["k"], gpu["v"], gpu["pq"], gpu["pk"], wl.window, wl.shift)
    binding.rib_set_path(binding.RIB_PATH_GENERIC if path == "generic" else binding.RIB_PATH_NONE)
    try:
        dq, dk, dv, dpq, dpk = binding.rib_window_attn_bwd_masked(gpu["q"], gpu["k"], gpu["v"], gpu["pq"], gpu["pk"], out, lse,
                                                                  gpu["dout"], wl.window, wl.shift)
        used = binding.rib_last_path()
    finally:
        binding.rib_set_path(binding.RIB_PATH_NONE)
    torch.cuda.synchronize()
    assert binding.rib_query_status() == 0
    assert used == (binding.RIB_PATH_SM100 if is_fast(wl, path) else binding.RIB_PATH_GENERIC)
    ref = msk.bwd(*(to_f64(cpu[k]) for k in ("q", "k", "v", "pq", "pk", "dout")), wl.window, wl.shift)
    for name, got, want in zip(("dq", "dk", "dv"), (dq, dk, dv), ref[:3]):
        compare(name, to_f64(got), want)
    scale = max(1.0, float(np.abs(ref[3]).max()), float(np.abs(ref[4]).max()))
    compare("dpq", to_f64(dpq), ref[3], max_abs=1e-2 * scale)
    compare("dpk", to_f64(dpk), ref[4], max_abs=1e-2 * scale)


def test_masked_keys_far_above_the_rest_do_not_disturb_the_rows_that_must_not_see_them():
    """The fast softmax form takes its reference from the first keys of the window, masked or not; keys of the wrapped
    part are scaled until their logits lie about 200 nat above the others: rows of the other part must still come
    out right (they are repaired by the exact form where the reference was out of range)."""
    wl = Workload("m_far", 1, 64, 64, 2, 32, 16, 32, 16, seed=92)
    cpu = synthetic.make_inputs(wl, with_dout=False)
    k = cpu["k"].clone()
    k[:, :16] = (k[:, :16].float() * 40.0).to(torch.bfloat16)          # image rows 0..15: the wrapped part of the last window row
    cpu["k"] = k
    gpu = {name: t.cuda() for name, t in cpu.items()}
    out, lse = binding.rib_window_attn_fwd_masked(gpu["q"], gpu["k"], gpu["v"], gpu["pq"], gpu["pk"], wl.window, wl.shift)
    torch.cuda.synchronize()
    assert binding.rib_query_status() == 0 and binding.rib_last_path() == binding.RIB_PATH_SM100
    ref_out, ref_lse = msk.fwd(*(to_f64(cpu[n]) for n in ("q", "k", "v", "pq", "pk")), wl.window, wl.shift)
    # rows that see the scaled keys are nearly one-hot: their output is one value row, up to 4.6 in size, stored as bf16
    # (spacing 2^-5 there), so the absolute bound is scaled by the size of the reference
    compare("out", to_f64(out), ref_out, max_abs=1e-2 * max(1.0, float(np.abs(ref_out).max()) / 2.0))
    compare("lse", to_f64(lse), ref_lse, max_abs=5e-2)      # logits of some hundred nat: fp32 carries them to a few 1e-5 relative


def test_masked_entry_points_reject_maps_the_window_does_not_divide():
    x = torch.zeros(40 * 56 * 32, dtype=torch.bfloat16, device="cuda")
    pos = torch.zeros(256 * 16, dtype=torch.bfloat16, device="cuda")
    rc = binding.library().rib_window_attn_fwd_masked(x.data_ptr(), x.data_ptr(), x.data_ptr(), pos.data_ptr(), pos.data_ptr(), 0,
                                                      1, 40, 56, 1, 32, 16, 16, 8, x.data_ptr(), None, None)
    assert rc == -2      # RIB_ERR_SHAPE

"""GPU parity: the CUDA path, called through the C ABI, against the CPU oracle on the same seeded
inputs, every element of every tensor, on the small cases and on the five benchmark configurations
at full size (the oracle needs a few seconds per configuration on the host cores)."""
import numpy as np
import pytest
import torch

from paper_2603_06738_b200 import binding, synthetic
from paper_2603_06738_b200.synthetic import CONFIGS, Workload

from parity_util import (compare, make, oracle_bwd, oracle_fwd, run_bwd, run_fwd, to_f64)

pytestmark = pytest.mark.gpu

# name, B, H, W, heads, d, r, window, shift
SMALL = [
    Workload("tiny_2x2", 2, 4, 4, 1, 8, 8, 2, 1, seed=11),
    Workload("w4_s2", 2, 8, 8, 2, 16, 8, 4, 2, seed=12),
    Workload("w8_s3_d32", 1, 16, 24, 3, 32, 16, 8, 3, seed=13),
    Workload("w6_ragged_rows", 1, 12, 18, 2, 24, 24, 6, 5, seed=14),       # n = 36: ragged row tile
    Workload("w20_ragged_tiles", 1, 40, 40, 2, 32, 16, 20, 7, seed=15),    # n = 400: several tiles + tail
    Workload("d64_r64", 1, 16, 16, 2, 64, 64, 8, 0, seed=16),
    Workload("rank0", 1, 16, 16, 2, 32, 0, 8, 4, seed=17),
    Workload("w16_s8_fast_shape", 2, 32, 48, 2, 32, 16, 16, 8, seed=18),   # fast-path shape, small
    Workload("w32_s16_fast_shape", 1, 64, 32, 3, 32, 16, 32, 16, seed=19),
    Workload("w48_s24_fast_shape", 1, 48, 96, 1, 32, 16, 48, 24, seed=20),
    Workload("w16_odd_shift", 1, 32, 32, 2, 32, 16, 16, 5, seed=21),       # fast shape but odd shift
    Workload("w16_s8_rank32", 2, 32, 48, 2, 32, 32, 16, 8, seed=22),       # rank 32 (d + r = 64) on the tcgen05 kernels
    Workload("w32_s16_rank32", 1, 64, 32, 3, 32, 32, 32, 16, seed=23),
    # the head widths of the paper's other network rows (appendix table of network implementations): 60-byte rows, which the
    # tcgen05 kernels take through zero-padded copies when d and r are even (r = 34: the two columns above 32 ride in the spare channels of d = 30)
    Workload("sst_d30_r18_w16", 1, 32, 32, 6, 30, 18, 16, 0, seed=24),
    Workload("sst_d30_r34_w32", 1, 32, 64, 3, 30, 34, 32, 16, seed=25),
    Workload("sst_d30_r18_w32_headwise", 2, 64, 32, 3, 30, 18, 32, 16, seed=36, headwise=True),   # zero-padded copies, tcgen05 kernels
    Workload("d10_r6_w16", 1, 32, 32, 2, 10, 6, 16, 8, seed=37),
    Workload("sst_d30_r34_w16_headwise", 2, 32, 48, 3, 30, 34, 16, 8, seed=38, headwise=True),   # rank 34: two columns ride in the head's spare channels
    Workload("light_d16_r24_w16", 2, 32, 32, 3, 16, 24, 16, 8, seed=26),       # d + r = 40: not a multiple of 16
    Workload("odd_d15_r7_w8", 1, 16, 16, 2, 15, 7, 8, 3, seed=27),
    # head widths and ranks that are multiples of 8: 32-wide tiles filled up with zeros by the TMA boxes (tcgen05 kernels)
    Workload("d16_r16_w32_s16", 1, 64, 32, 3, 16, 16, 32, 16, seed=28),
    Workload("d24_r8_w16_s8", 2, 32, 48, 2, 24, 8, 16, 8, seed=29),
    Workload("d8_r32_w16", 1, 32, 32, 2, 8, 32, 16, 0, seed=30),
    Workload("d16_r24_w32_headwise", 1, 32, 64, 3, 16, 24, 32, 8, seed=31, headwise=True),
    # windows of 8 x 8 tokens (half a tile): worked as 16 x 16 windows that hold 2 x 2 of them on the tcgen05 kernels
    Workload("w8_packed", 2, 32, 48, 3, 32, 16, 8, 0, seed=32),
    Workload("w8_packed_rank32_headwise", 1, 16, 32, 2, 32, 32, 8, 0, seed=33, headwise=True),
    Workload("w8_packed_d16_r24", 1, 32, 32, 4, 16, 24, 8, 0, seed=34),
    Workload("w8_rows_24", 1, 24, 32, 2, 32, 16, 8, 0, seed=35),               # 24 rows: not a multiple of 16, any-shape kernels
]
NARROW = [wl for wl in SMALL if wl.name in ("light_d16_r24_w16", "d16_r16_w32_s16", "d24_r8_w16_s8", "d8_r32_w16", "d16_r24_w32_headwise",
                                             "w8_packed", "w8_packed_rank32_headwise", "w8_packed_d16_r24",
                                             "sst_d30_r18_w16", "sst_d30_r18_w32_headwise", "d10_r6_w16", "sst_d30_r34_w32", "sst_d30_r34_w16_headwise")]


def _inputs_for(wl):
    if wl.r == 0:
        cpu = synthetic.make_inputs(Workload(wl.name, wl.B, wl.H, wl.W, wl.heads, wl.d, 8, wl.window, wl.shift, wl.seed), True)
        cpu["pq"] = cpu["pq"][:, :0].contiguous()
        cpu["pk"] = cpu["pk"][:, :0].contiguous()
        return cpu, {k: v.cuda() for k, v in cpu.items()}
    return make(wl, with_dout=True)


@pytest.mark.parametrize("wl", SMALL, ids=lambda w: w.name)
@pytest.mark.parametrize("path", ["auto", "generic"])
def test_small_forward_and_backward_every_element(wl, path):
    cpu, gpu = _inputs_for(wl)
    binding.rib_set_path(binding.RIB_PATH_GENERIC if path == "generic" else binding.RIB_PATH_NONE)
    try:
        out, lse = run_fwd(gpu, wl)
        fwd_path = binding.rib_last_path()
        dq, dk, dv, dpq, dpk = run_bwd(gpu, wl, out, lse)
    finally:
        binding.rib_set_path(binding.RIB_PATH_NONE)
    if path == "generic":
        assert fwd_path == binding.RIB_PATH_GENERIC
    ref_out, ref_lse = oracle_fwd(cpu, wl)
    compare("out", to_f64(out), ref_out)
    compare("lse", to_f64(lse), ref_lse)
    rdq, rdk, rdv, rdpq, rdpk = oracle_bwd(cpu, wl)
    # A window of 64 tokens averages over few keys: gradients reach 2 in size where those of the benchmark windows stay
    # below 1.3, and a bf16 result of that size is spaced 2^-7 apart.  The absolute bound follows the size of the
    # reference there; the relative-L2 bound is the same everywhere.
    grad_abs = 1e-2 * max(1.0, float(np.abs(rdq).max()), float(np.abs(rdk).max())) if wl.window == 8 else 1e-2
    compare("dq", to_f64(dq), rdq, max_abs=grad_abs)
    compare("dk", to_f64(dk), rdk, max_abs=grad_abs)
    compare("dv", to_f64(dv), rdv)
    if wl.r:
        # sums over every pair of the batch: bounded relative to the largest entry, as in the full-size tests
        scale = max(1.0, float(np.abs(rdpq).max()), float(np.abs(rdpk).max()))
        compare("dpq", to_f64(dpq), rdpq, max_abs=1e-2 * scale)
        compare("dpk", to_f64(dpk), rdpk, max_abs=1e-2 * scale)


@pytest.mark.parametrize("wl", NARROW, ids=lambda w: w.name)
def test_narrow_heads_and_ranks_take_the_tcgen05_kernels(wl):
    """d = 8, 16, 24, r = 8, 16, 24, 32 and windows of 8 x 8 tokens run on the tensor-core kernels (the parity of these
    shapes is checked above)."""
    _, gpu = _inputs_for(wl)
    out, lse = run_fwd(gpu, wl)
    assert binding.rib_last_path() == binding.RIB_PATH_SM100
    run_bwd(gpu, wl, out, lse)
    assert binding.rib_last_path() == binding.RIB_PATH_SM100


def test_lse_is_optional_and_outputs_are_fully_written():
    wl = SMALL[2]
    cpu, gpu = make(wl)
    out = torch.full_like(gpu["q"], float("nan"))
    binding.rib_window_attn_fwd(gpu["q"], gpu["k"], gpu["v"], gpu["pq"], gpu["pk"], wl.window, wl.shift,
                                out=out, want_lse=False)
    torch.cuda.synchronize()
    assert torch.isfinite(out.float()).all()
    ref_out, _ = oracle_fwd(cpu, wl)
    compare("out", to_f64(out), ref_out)


def test_config1_full_forward():
    wl = CONFIGS[0]
    cpu, gpu = make(wl, with_dout=False)
    out, lse = run_fwd(gpu, wl)
    ref_out, ref_lse = oracle_fwd(cpu, wl)
    compare("out", to_f64(out), ref_out)
    compare("lse", to_f64(lse), ref_lse)


@pytest.mark.parametrize("idx", [1, 2, 3])
def test_full_size_forward_all_pairs(idx):
    """Benchmark configurations 2-4 at full size, in the launch configuration the benchmark times: every pair
    against the oracle."""
    wl = CONFIGS[idx]
    cpu, gpu = make(wl, with_dout=False)
    out, lse = run_fwd(gpu, wl)
    assert binding.rib_last_path() == binding.RIB_PATH_SM100
    ref_out, ref_lse = oracle_fwd(cpu, wl)
    compare(f"cfg{idx + 1} out", to_f64(out), ref_out)
    compare(f"cfg{idx + 1} lse", to_f64(lse), ref_lse)


def _full_forward_backward_all_pairs(wl, tag):
    cpu, gpu = make(wl, with_dout=True)
    out, lse = run_fwd(gpu, wl)
    assert binding.rib_last_path() == binding.RIB_PATH_SM100
    dq, dk, dv, dpq, dpk = run_bwd(gpu, wl, out, lse)
    assert binding.rib_last_path() == binding.RIB_PATH_SM100
    ref_out, ref_lse = oracle_fwd(cpu, wl)
    compare(f"{tag} out", to_f64(out), ref_out)
    compare(f"{tag} lse", to_f64(lse), ref_lse)
    rdq, rdk, rdv, rdpq, rdpk = oracle_bwd(cpu, wl)
    compare(f"{tag} dq", to_f64(dq), rdq)
    compare(f"{tag} dk", to_f64(dk), rdk)
    compare(f"{tag} dv", to_f64(dv), rdv)
    # dPq/dPk are sums over pairs * n terms of magnitude ~1 and grow with the problem (max|ref| is printed): their
    # absolute bound is 1e-2 relative to the largest entry, the relative-L2 bound is the unscaled 5e-3.
    scale = max(1.0, float(np.abs(rdpq).max()), float(np.abs(rdpk).max()))
    compare(f"{tag} dpq", to_f64(dpq), rdpq, max_abs=1e-2 * scale)
    compare(f"{tag} dpk", to_f64(dpk), rdpk, max_abs=1e-2 * scale)


def test_config5_full_forward_backward_all_pairs():
    """Training configuration at full size: out, lse, dq, dk, dv, dPq, dPk over every pair."""
    _full_forward_backward_all_pairs(CONFIGS[4], "cfg5")


def test_rank32_full_size_forward_and_backward_all_pairs():
    """The paper's second window cycle uses rank 32 with 32-channel heads (d + r = 64): both passes run on the
    tcgen05 kernels (64-byte RIB rows; dK~ and dQ~ 64 columns wide), checked at the training-patch size on every pair."""
    base = CONFIGS[1]
    _full_forward_backward_all_pairs(
        Workload("cfg2_rank32", base.B, base.H, base.W, base.heads, base.d, 32, base.window, base.shift, seed=34), "cfg2 r32")


def test_largest_paper_window_96_forward_and_backward():
    """The paper's largest attention window (96 x 96 = 9216 tokens per window, 72 key blocks): the
    whole 96 x 96 map is one shifted window per head."""
    wl = Workload("w96_s48", 1, 96, 96, 2, 32, 16, 96, 48, seed=33)
    cpu, gpu = make(wl, with_dout=True)
    out, lse = run_fwd(gpu, wl)
    assert binding.rib_last_path() == binding.RIB_PATH_SM100
    dq, dk, dv, dpq, dpk = run_bwd(gpu, wl, out, lse)
    assert binding.rib_last_path() == binding.RIB_PATH_SM100
    ref_out, ref_lse = oracle_fwd(cpu, wl)
    compare("out", to_f64(out), ref_out)
    compare("lse", to_f64(lse), ref_lse)
    rdq, rdk, rdv, rdpq, rdpk = oracle_bwd(cpu, wl)
    compare("dq", to_f64(dq), rdq)
    compare("dk", to_f64(dk), rdk)
    compare("dv", to_f64(dv), rdv)
    compare("dpq", to_f64(dpq), rdpq)
    compare("dpk", to_f64(dpk), rdpk)


@pytest.mark.parametrize("direction", ["growing", "shrinking"])
def test_running_maximum_rescale(direction):
    """Logits that grow (or shrink) steeply along the key order force the online-softmax rescale
    of the accumulated output in later key blocks."""
    wl = Workload("w32_rescale", 1, 32, 64, 2, 32, 16, 32, 0, seed=31)
    cpu, gpu = make(wl, with_dout=False)
    ramp = torch.linspace(0.2, 6.0, wl.H).view(1, wl.H, 1, 1, 1)
    if direction == "shrinking":
        ramp = ramp.flip(1)
    cpu["k"] = (cpu["k"].float() * ramp).to(torch.bfloat16)      # |k| grows with the row of the window
    cpu["q"] = (cpu["q"].float() * 2.0).to(torch.bfloat16)
    gpu = {k: v.cuda() for k, v in cpu.items()}
    out, lse = run_fwd(gpu, wl)
    assert binding.rib_last_path() == binding.RIB_PATH_SM100
    ref_out, ref_lse = oracle_fwd(cpu, wl)
    assert np.abs(ref_lse).max() > 20          # the case really has large logits
    compare("out", to_f64(out), ref_out, max_abs=2e-2)
    compare("lse", to_f64(lse), ref_lse, max_abs=2e-2, rel_l2=5e-3)


@pytest.mark.parametrize("wl", [SMALL[7], SMALL[8], SMALL[12], CONFIGS[1]] + [w for w in SMALL if w.name in ("w8_packed", "d16_r16_w32_s16")],
                         ids=lambda w: w.name)
def test_exact_softmax_form_every_element(wl):
    """The tcgen05 forward kernel keeps two forms of the softmax: a fast one with a fixed per-row reference and the
    exact one with a running maximum that redoes items whose scores leave the fast form's range.  Here every item is
    forced through the exact form."""
    cpu, gpu = make(wl, with_dout=False)
    binding.rib_set_path(binding.RIB_PATH_SM100_EXACT)
    try:
        out, lse = run_fwd(gpu, wl)
        assert binding.rib_last_path() == binding.RIB_PATH_SM100
    finally:
        binding.rib_set_path(binding.RIB_PATH_NONE)
    ref_out, ref_lse = oracle_fwd(cpu, wl)
    compare("out (exact form)", to_f64(out), ref_out)
    compare("lse (exact form)", to_f64(lse), ref_lse)


@pytest.mark.parametrize("where", ["late_key", "first_key"])
def test_scores_beyond_the_fast_softmax_range_are_redone_exactly(where):
    """One key of every window is scaled until its logits lie ~ +-200 nat from the rest: rows that like it are one-hot
    on it, rows that dislike it see it 200 nat below their reference.  Both leave what a fixed reference can
    represent in fp32 (about +-85 nat); the kernel must notice and redo those items with the running maximum."""
    wl = Workload("w32_far_scores", 2, 64, 64, 2, 32, 16, 32, 16, seed=35)
    cpu, gpu = make(wl, with_dout=False)
    k = cpu["k"].float()
    y, x = (40, 13) if where == "late_key" else (wl.shift, wl.shift)       # (shift, shift) is token 0 of window (0, 0)
    for yy in range(y % wl.window, wl.H, wl.window):
        for xx in range(x % wl.window, wl.W, wl.window):
            k[:, yy, xx] *= 220.0
    cpu["k"] = k.to(torch.bfloat16)
    gpu = {kk: v.cuda() for kk, v in cpu.items()}
    out, lse = run_fwd(gpu, wl)
    assert binding.rib_last_path() == binding.RIB_PATH_SM100
    ref_out, ref_lse = oracle_fwd(cpu, wl)
    assert np.abs(ref_lse).max() > 150          # the case really leaves the range
    compare("out", to_f64(out), ref_out, max_abs=2e-2)
    compare("lse", to_f64(lse), ref_lse, max_abs=2e-2 * max(1.0, np.abs(ref_lse).max() / 100))


def test_fast_path_is_taken_for_benchmark_shapes():
    for wl in CONFIGS:
        small = Workload(wl.name, 1, wl.window, wl.window, 1, wl.d, wl.r, wl.window, wl.shift, seed=1)
        cpu, gpu = make(small, with_dout=False)
        out, lse = run_fwd(gpu, small)
        assert binding.rib_last_path() == binding.RIB_PATH_SM100, wl.name
        gpu["dout"] = torch.ones_like(out)
        run_bwd(gpu, small, out, lse)
        assert binding.rib_last_path() == binding.RIB_PATH_SM100, wl.name


def test_outputs_do_not_depend_on_stale_memory():
    """Two calls in a row on the same buffers (and the same workspace) give the same bits for
    out/lse/dk/dv; dq, dPq and dPk are fp32 sums whose order may differ from run to run."""
    wl = SMALL[7]
    cpu, gpu = make(wl)
    out1, lse1 = run_fwd(gpu, wl)
    out2, lse2 = run_fwd(gpu, wl)
    assert torch.equal(out1, out2) and torch.equal(lse1, lse2)
    need = binding.rib_window_attn_bwd_workspace(wl.B, wl.H, wl.W, wl.heads, wl.d, wl.r, wl.window)
    workspace = torch.full((need,), 0x7f, dtype=torch.uint8, device="cuda")     # stale, non-zero scratch
    a = binding.rib_window_attn_bwd(gpu["q"], gpu["k"], gpu["v"], gpu["pq"], gpu["pk"], out1, lse1, gpu["dout"],
                                    wl.window, wl.shift, workspace=workspace)
    b = binding.rib_window_attn_bwd(gpu["q"], gpu["k"], gpu["v"], gpu["pq"], gpu["pk"], out1, lse1, gpu["dout"],
                                    wl.window, wl.shift, workspace=workspace)
    torch.cuda.synchronize()
    assert binding.rib_query_status() == 0
    assert binding.rib_last_path() == binding.RIB_PATH_SM100
    for x, y in zip(a[1:3], b[1:3]):
        assert torch.equal(x, y)
    torch.testing.assert_close(a[0].float(), b[0].float(), rtol=2e-2, atol=1e-3)
    for x, y in zip(a[3:], b[3:]):
        torch.testing.assert_close(x, y, rtol=1e-4, atol=1e-4)

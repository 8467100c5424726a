"""GPU parity for head-wise positional features (Sec. 3.1, the remark after Eq. 3: one Pq / Pk
table per head): the `_headwise` entry points against the CPU oracle called with [heads, n, r]
tables, on both kernel families, plus the relations that tie them to the shared-table calls."""
import ctypes

import numpy as np
import pytest
import torch

from paper_2603_06738_b200 import binding
from paper_2603_06738_b200.synthetic import CONFIGS, Workload

from parity_util import (compare, make, oracle_bwd, oracle_fwd, run_bwd, run_fwd, to_f64)

pytestmark = pytest.mark.gpu

HEADWISE = [
    Workload("hw_w4_generic", 2, 8, 8, 3, 16, 8, 4, 2, seed=41, headwise=True),
    Workload("hw_w20_ragged", 1, 40, 40, 2, 32, 16, 20, 7, seed=42, headwise=True),
    Workload("hw_w16_s8", 2, 32, 48, 3, 32, 16, 16, 8, seed=43, headwise=True),      # 12 windows per head
    Workload("hw_w32_s16", 1, 64, 64, 6, 32, 16, 32, 16, seed=44, headwise=True),    # 4 windows per head
    Workload("hw_w48_one_window", 1, 48, 48, 5, 32, 16, 48, 24, seed=45, headwise=True),
    Workload("hw_w16_rank32", 1, 32, 32, 3, 32, 32, 16, 8, seed=49, headwise=True),   # rank 32 (d + r = 64)
]


@pytest.mark.parametrize("wl", HEADWISE, ids=lambda w: w.name)
@pytest.mark.parametrize("path", ["auto", "generic"])
def test_headwise_forward_and_backward_every_element(wl, path):
    cpu, gpu = make(wl, with_dout=True)
    binding.rib_set_path(binding.RIB_PATH_GENERIC if path == "generic" else binding.RIB_PATH_NONE)
    try:
        out, lse = run_fwd(gpu, wl)
        fwd_path = binding.rib_last_path()
        dq, dk, dv, dpq, dpk = run_bwd(gpu, wl, out, lse)
        bwd_path = binding.rib_last_path()
    finally:
        binding.rib_set_path(binding.RIB_PATH_NONE)
    fast_shape = wl.d == 32 and wl.window % 16 == 0 and wl.shift % 8 == 0
    fast = {True: binding.RIB_PATH_SM100, False: binding.RIB_PATH_GENERIC}
    expected = fast[path == "auto" and fast_shape and wl.r in (16, 32)]
    assert fwd_path == expected and bwd_path == expected
    ref_out, ref_lse = oracle_fwd(cpu, wl)
    compare("out", to_f64(out), ref_out)
    compare("lse", to_f64(lse), ref_lse)
    rdq, rdk, rdv, rdpq, rdpk = oracle_bwd(cpu, wl)
    assert rdpq.shape == (wl.heads, wl.n, wl.r)
    compare("dq", to_f64(dq), rdq)
    compare("dk", to_f64(dk), rdk)
    compare("dv", to_f64(dv), rdv)
    for h in range(wl.heads):   # head by head: a table written to the wrong head fails here
        compare(f"dpq[{h}]", to_f64(dpq[h]), rdpq[h])
        compare(f"dpk[{h}]", to_f64(dpk[h]), rdpk[h])


def test_equal_tables_reproduce_the_shared_call():
    """With the same table in every head the forward results are those of the shared-table call bit
    for bit, and the head-wise gradients add up to the shared ones."""
    wl = Workload("hw_equal_tables", 2, 64, 32, 3, 32, 16, 32, 8, seed=46)
    cpu, gpu = make(wl, with_dout=True)
    out, lse = run_fwd(gpu, wl)
    dq, dk, dv, dpq, dpk = run_bwd(gpu, wl, out, lse)
    pq_h = gpu["pq"].unsqueeze(0).repeat(wl.heads, 1, 1).contiguous()
    pk_h = gpu["pk"].unsqueeze(0).repeat(wl.heads, 1, 1).contiguous()
    out_h, lse_h = binding.rib_window_attn_fwd_headwise(gpu["q"], gpu["k"], gpu["v"], pq_h, pk_h, wl.window, wl.shift)
    res_h = binding.rib_window_attn_bwd_headwise(gpu["q"], gpu["k"], gpu["v"], pq_h, pk_h, out, lse, gpu["dout"],
                                                 wl.window, wl.shift)
    torch.cuda.synchronize()
    assert binding.rib_query_status() == 0
    assert torch.equal(out_h, out) and torch.equal(lse_h, lse)
    assert torch.equal(res_h[1], dk) and torch.equal(res_h[2], dv)
    # dq is summed over key blocks with atomic adds: equal up to the order of those additions
    compare("dq", to_f64(res_h[0]), to_f64(dq), max_abs=2e-3, rel_l2=1e-3)
    scale = max(1.0, float(dpq.abs().max()), float(dpk.abs().max()))
    compare("sum over heads of dpq", to_f64(res_h[3].sum(0)), to_f64(dpq), max_abs=1e-3 * scale, rel_l2=1e-4)
    compare("sum over heads of dpk", to_f64(res_h[4].sum(0)), to_f64(dpk), max_abs=1e-3 * scale, rel_l2=1e-4)


@pytest.mark.parametrize("path", ["auto", "generic"])
def test_padded_head_stride_through_the_c_abi(path):
    """Tables further apart than n * r elements: the gaps are never read (they hold NaN) and the
    results equal those of the packed layout."""
    wl = Workload("hw_padded", 1, 32, 32, 3, 32, 16, 16, 8, seed=47, headwise=True)
    cpu, gpu = make(wl, with_dout=True)
    out, lse = run_fwd(gpu, wl)
    packed = run_bwd(gpu, wl, out, lse)
    n, r, heads = wl.n, wl.r, wl.heads
    stride = n * r + 64
    nan = float("nan")
    pq_p = torch.full((heads, stride), nan, dtype=torch.bfloat16, device="cuda")
    pk_p = torch.full((heads, stride), nan, dtype=torch.bfloat16, device="cuda")
    pq_p[:, :n * r] = gpu["pq"].reshape(heads, -1)
    pk_p[:, :n * r] = gpu["pk"].reshape(heads, -1)
    out_p, lse_p = torch.empty_like(out), torch.empty_like(lse)
    dq, dk, dv = (torch.empty_like(out) for _ in range(3))
    dpq = torch.full((heads, stride), nan, dtype=torch.float32, device="cuda")
    dpk = torch.full((heads, stride), nan, dtype=torch.float32, device="cuda")
    lib = binding.library()
    B, H, W, d = wl.B, wl.H, wl.W, wl.d
    need = lib.rib_window_attn_bwd_headwise_workspace(stride, B, H, W, heads, d, r, wl.window)
    ws = torch.empty(max(need, 256), dtype=torch.uint8, device="cuda")
    st = torch.cuda.current_stream().cuda_stream
    binding.rib_set_path(binding.RIB_PATH_GENERIC if path == "generic" else binding.RIB_PATH_NONE)
    try:
        rc = lib.rib_window_attn_fwd_headwise(gpu["q"].data_ptr(), gpu["k"].data_ptr(), gpu["v"].data_ptr(),
                                              pq_p.data_ptr(), pk_p.data_ptr(), stride, B, H, W, heads, d, r, wl.window,
                                              wl.shift, out_p.data_ptr(), lse_p.data_ptr(), st)
        assert rc == 0
        rc = lib.rib_window_attn_bwd_headwise(gpu["q"].data_ptr(), gpu["k"].data_ptr(), gpu["v"].data_ptr(),
                                              pq_p.data_ptr(), pk_p.data_ptr(), stride, out.data_ptr(), lse.data_ptr(),
                                              gpu["dout"].data_ptr(), B, H, W, heads, d, r, wl.window, wl.shift,
                                              dq.data_ptr(), dk.data_ptr(), dv.data_ptr(), dpq.data_ptr(), dpk.data_ptr(),
                                              ws.data_ptr(), ws.numel(), st)
        assert rc == 0
    finally:
        binding.rib_set_path(binding.RIB_PATH_NONE)
    torch.cuda.synchronize()
    assert binding.rib_query_status() == 0
    if path == "auto":
        assert torch.equal(out_p, out) and torch.equal(lse_p, lse)
        assert torch.equal(dk, packed[1]) and torch.equal(dv, packed[2])
    ref = oracle_bwd(cpu, wl)
    compare("out", to_f64(out_p), oracle_fwd(cpu, wl)[0])
    compare("dq", to_f64(dq), ref[0])
    compare("dpq", to_f64(dpq[:, :n * r]).reshape(heads, n, r), ref[3])
    compare("dpk", to_f64(dpk[:, :n * r]).reshape(heads, n, r), ref[4])


def test_bad_head_stride_is_rejected_before_any_launch():
    lib = binding.library()
    x = torch.zeros(1024, dtype=torch.uint8, device="cuda")
    ptr = x.data_ptr()
    launches = binding.rib_kernel_launches()
    for stride in (16 * 16 * 16 - 8, 16 * 16 * 16 + 4, -4096):   # too small, not a multiple of 8, negative
        rc = lib.rib_window_attn_fwd_headwise(ptr, ptr, ptr, ptr, ptr, stride, 1, 16, 16, 2, 32, 16, 16, 0, ptr, None,
                                              None)
        assert rc == -2, stride   # RIB_ERR_SHAPE
        assert lib.rib_window_attn_bwd_headwise_workspace(stride, 1, 16, 16, 2, 32, 16, 16) == 0
    assert binding.rib_kernel_launches() == launches


def test_training_shape_full_size_headwise():
    """The training configuration with head-wise tables at full size, every pair: out, lse, dq, dk, dv and
    the per-head dPq/dPk reductions."""
    base = CONFIGS[4]
    wl = Workload("cfg5_headwise", base.B, base.H, base.W, base.heads, base.d, base.r, base.window, base.shift,
                  seed=48, backward=True, headwise=True)
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
    scale = max(1.0, float(np.abs(rdpq).max()), float(np.abs(rdpk).max()))
    for h in range(wl.heads):
        compare(f"dpq[{h}]", to_f64(dpq[h]), rdpq[h], max_abs=1e-2 * scale)
        compare(f"dpk[{h}]", to_f64(dpk[h]), rdpk[h], max_abs=1e-2 * scale)

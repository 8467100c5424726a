"""The backward entry point that brings its own scratch memory (for callers that may not allocate
on the device) gives the same gradients as the entry point that takes a caller's workspace.

Collected last on purpose (file name): a run that stops at the first failure has then already run
every other test.  The test does not depend on what ran before it: the built-in scratch is shared
by all calls and keeps the previous call's contents, which is exactly what two calls in a row
exercise."""
import pytest
import torch

from paper_2603_06738_b200 import binding
from paper_2603_06738_b200.synthetic import Workload

from parity_util import compare, make, oracle_bwd, run_bwd, run_fwd, to_f64

pytestmark = pytest.mark.gpu


def _noalloc_bwd(gpu, wl, out, lse):
    """Results are pre-filled with NaN so that anything the call leaves unwritten shows up."""
    dq, dk, dv = (torch.full_like(gpu["q"], float("nan")) for _ in range(3))
    dpq, dpk = (torch.full((wl.n, wl.r), float("nan"), dtype=torch.float32, device="cuda") for _ in range(2))
    binding.rib_window_attn_bwd_noalloc(gpu["q"], gpu["k"], gpu["v"], gpu["pq"], gpu["pk"], out, lse, gpu["dout"],
                                        dq, dk, dv, dpq, dpk, wl.window, wl.shift)
    torch.cuda.synchronize()
    assert binding.rib_query_status() == 0
    return dq, dk, dv, dpq, dpk


@pytest.mark.parametrize("wl", [
    Workload("noalloc_w16_s8", 2, 32, 48, 2, 32, 16, 16, 8, seed=41),      # tcgen05 kernels
    Workload("noalloc_w6_s5", 1, 12, 18, 2, 24, 24, 6, 5, seed=42),        # any-shape kernels
], ids=lambda w: w.name)
def test_noalloc_backward_matches_workspace_backward_twice(wl):
    cpu, gpu = make(wl, with_dout=True)
    out, lse = run_fwd(gpu, wl)
    ref = run_bwd(gpu, wl, out, lse)
    ref_path = binding.rib_last_path()
    want = oracle_bwd(cpu, wl)        # the gradients the paper's definition gives (CPU oracle)
    for attempt in range(2):      # the second call finds the first call's leftovers in the scratch
        if attempt == 1:
            # what the entry point is for: once its scratch address is known (first call), a call takes no device memory
            dq, dk, dv = (torch.empty_like(gpu["q"]) for _ in range(3))
            dpq, dpk = (torch.empty((wl.n, wl.r), dtype=torch.float32, device="cuda") for _ in range(2))
            torch.cuda.synchronize()
            free_before = torch.cuda.mem_get_info()[0]
            binding.rib_window_attn_bwd_noalloc(gpu["q"], gpu["k"], gpu["v"], gpu["pq"], gpu["pk"], out, lse, gpu["dout"],
                                                dq, dk, dv, dpq, dpk, wl.window, wl.shift)
            torch.cuda.synchronize()
            assert torch.cuda.mem_get_info()[0] == free_before, "the call changed the device's free memory"
        got = _noalloc_bwd(gpu, wl, out, lse)
        assert binding.rib_last_path() == ref_path
        for name, x, y in zip(("dq", "dk", "dv", "dpq", "dpk"), got, ref):
            assert torch.isfinite(x.float()).all(), f"{name} (call {attempt}) has unwritten or non-finite values"
            # same kernels on the same inputs: only the order of the fp32 atomic sums may differ
            torch.testing.assert_close(x.float(), y.float(), rtol=2e-2, atol=1e-3, msg=lambda m: f"{name}: {m}")
        for name, x, r in zip(("dq", "dk", "dv", "dpq", "dpk"), got, want):
            scale = max(1.0, float(abs(r).max())) if name in ("dpq", "dpk") else 1.0      # sums over all pairs: bound relative to their size
            compare(f"{name} (call {attempt}, against the oracle)", to_f64(x), r, max_abs=1e-2 * scale)


def test_noalloc_rejects_shapes_beyond_the_builtin_scratch():
    B, H, W, heads, d, r, window = 16, 96, 96, 6, 32, 16, 32
    assert binding.rib_window_attn_bwd_workspace(B, H, W, heads, d, r, window) > binding.RIB_NOALLOC_SCRATCH_BYTES
    lib = binding.library()
    fake = [256 * (i + 1) for i in range(13)]       # never dereferenced: the size check comes first
    rc = lib.rib_window_attn_bwd_noalloc(*fake[:8], B, H, W, heads, d, r, window, 0, *fake[8:], None)
    assert rc == -8 and "TOO_LARGE" in binding.rib_status_string(rc)

"""Safety nets that stand in for a memory checker and for fault injection:

* the give-up path of the bounded device-side waits is exercised by a self-test kernel whose wait
  really runs out (nothing is made to fault or hang: the kernel returns by itself after the limit);
* every output and the workspace are placed between guard bands of a known byte pattern, which must
  be intact after the call, and the outputs are pre-filled with NaN so that unwritten parts show."""
import numpy as np
import pytest
import torch

from paper_2603_06738_b200 import binding, synthetic
from paper_2603_06738_b200.synthetic import Workload

from parity_util import compare, make, oracle_bwd, oracle_fwd, run_fwd, to_f64

pytestmark = pytest.mark.gpu

GUARD = 4096
PATTERN = 0xA5


def test_a_wait_that_runs_out_reports_and_leaves_the_device_usable():
    assert binding.rib_query_status() == 0
    binding.rib_wait_probe(1_000_000)          # 1 ms
    torch.cuda.synchronize()
    assert binding.rib_query_status() == binding.RIB_ERR_DEVICE_WAIT
    assert binding.rib_query_status() == 0     # reading clears the word
    # tensor memory was handed back and the context is intact: a normal forward call passes parity straight after
    wl = Workload("after_timeout_w16_s8", 2, 32, 48, 2, 32, 16, 16, 8, seed=61)
    cpu, gpu = make(wl, with_dout=False)
    out, lse = run_fwd(gpu, wl)
    assert binding.rib_last_path() == binding.RIB_PATH_SM100
    ref_out, ref_lse = oracle_fwd(cpu, wl)
    compare("out", to_f64(out), ref_out)
    compare("lse", to_f64(lse), ref_lse)
    # limits outside 1 ns .. 0.1 s are refused without a launch
    launches = binding.rib_kernel_launches()
    assert binding.library().rib_wait_probe(0, None) == -2
    assert binding.library().rib_wait_probe(10**9, None) == -2
    assert binding.rib_kernel_launches() == launches


class Guarded:
    """Tensors carved out of one byte buffer, each with GUARD bytes of PATTERN on both sides."""

    def __init__(self):
        self.regions = []

    def tensor(self, shape, dtype, fill=float("nan")):
        nbytes = int(np.prod(shape)) * torch.empty((), dtype=dtype).element_size()
        padded = (nbytes + 255) // 256 * 256
        raw = torch.full((GUARD + padded + GUARD,), PATTERN, dtype=torch.uint8, device="cuda")
        assert raw.data_ptr() % 256 == 0
        body = raw[GUARD:GUARD + nbytes].view(dtype).view(*shape)
        if dtype == torch.uint8:
            body.fill_(0x7F)
        else:
            body.fill_(fill)
        self.regions.append((raw, nbytes))
        return body

    def check(self, what):
        for i, (raw, nbytes) in enumerate(self.regions):
            front, back = raw[:GUARD], raw[GUARD + nbytes:]
            assert bool((front == PATTERN).all()) and bool((back == PATTERN).all()), f"{what}: guard band of buffer {i} was written"


SHAPES = [
    Workload("guard_w16_s8", 2, 32, 48, 2, 32, 16, 16, 8, seed=62),            # tcgen05 kernels
    Workload("guard_w32_rank32", 1, 64, 32, 3, 32, 32, 32, 16, seed=63),       # tcgen05 kernels, rank 32
    Workload("guard_w6_s5", 1, 12, 18, 2, 24, 24, 6, 5, seed=64),              # any-shape kernels
]


@pytest.mark.parametrize("wl", SHAPES, ids=lambda w: w.name)
def test_forward_and_backward_stay_inside_their_buffers(wl):
    cpu, gpu = make(wl, with_dout=True)
    g = Guarded()
    out = g.tensor(gpu["q"].shape, torch.bfloat16)
    lse = g.tensor((wl.B, wl.heads, wl.H, wl.W), torch.float32)
    binding.rib_window_attn_fwd(gpu["q"], gpu["k"], gpu["v"], gpu["pq"], gpu["pk"], wl.window, wl.shift, out=out, lse=lse)
    torch.cuda.synchronize()
    assert binding.rib_query_status() == 0
    g.check("forward")
    ref_out, ref_lse = oracle_fwd(cpu, wl)
    compare("out", to_f64(out), ref_out)
    compare("lse", to_f64(lse), ref_lse)

    # backward through the C ABI with guarded results and a guarded workspace
    g = Guarded()
    dq, dk, dv = (g.tensor(gpu["q"].shape, torch.bfloat16) for _ in range(3))
    dpq, dpk = (g.tensor((wl.n, wl.r), torch.float32) for _ in range(2))
    need = binding.rib_window_attn_bwd_workspace(wl.B, wl.H, wl.W, wl.heads, wl.d, wl.r, wl.window)
    ws = g.tensor((max(need, 256),), torch.uint8)
    P = lambda t: t.data_ptr()
    rc = binding.library().rib_window_attn_bwd(
        P(gpu["q"]), P(gpu["k"]), P(gpu["v"]), P(gpu["pq"]), P(gpu["pk"]), P(out), P(lse), P(gpu["dout"]),
        wl.B, wl.H, wl.W, wl.heads, wl.d, wl.r, wl.window, wl.shift, P(dq), P(dk), P(dv), P(dpq), P(dpk),
        P(ws), ws.numel(), None)
    assert rc == 0
    torch.cuda.synchronize()
    assert binding.rib_query_status() == 0
    g.check("backward")
    ref = oracle_bwd(cpu, wl)
    for name, got, want in zip(("dq", "dk", "dv", "dpq", "dpk"), (dq, dk, dv, dpq, dpk), ref):
        scale = max(1.0, float(np.abs(want).max())) if name in ("dpq", "dpk") else 1.0
        compare(name, to_f64(got), want, max_abs=1e-2 * scale)


def test_partial_window_and_gated_forward_stay_inside_their_buffers():
    lib = binding.library()
    P = lambda t: t.data_ptr()
    # a map that is not a multiple of the window (tcgen05 kernels: H, W multiples of 8)
    wl = Workload("guard_partial", 1, 40, 56, 2, 32, 16, 16, 8, seed=65)
    cpu, gpu = make(wl, with_dout=False)
    ref_out, ref_lse = binding.rib_window_attn_fwd_padded(gpu["q"], gpu["k"], gpu["v"], gpu["pq"], gpu["pk"], wl.window, wl.shift)
    g = Guarded()
    out = g.tensor(gpu["q"].shape, torch.bfloat16)
    lse = g.tensor((wl.B, wl.heads, wl.H, wl.W), torch.float32)
    rc = lib.rib_window_attn_fwd_padded(P(gpu["q"]), P(gpu["k"]), P(gpu["v"]), P(gpu["pq"]), P(gpu["pk"]), 0, wl.B, wl.H, wl.W,
                                        wl.heads, wl.d, wl.r, wl.window, wl.shift, P(out), P(lse), None)
    assert rc == 0
    torch.cuda.synchronize()
    assert binding.rib_query_status() == 0
    g.check("forward on partial windows")
    assert torch.equal(out, ref_out) and torch.equal(lse, ref_lse)
    # output multiplied by a gate (Eq. 9)
    wl = Workload("guard_gated", 1, 32, 32, 2, 32, 16, 16, 8, seed=66)
    cpu, gpu = make(wl, with_dout=False)
    gate = synthetic.bf16_tensor(66, "gate", (wl.B, wl.H, wl.W, wl.heads * wl.d), 0.3).abs().clamp(max=1.0).to(torch.bfloat16).cuda()
    ref_out, ref_lse = binding.rib_window_attn_fwd_gated(gpu["q"], gpu["k"], gpu["v"], gpu["pq"], gpu["pk"], gate, wl.window, wl.shift)
    g = Guarded()
    out = g.tensor(gpu["q"].shape, torch.bfloat16)
    lse = g.tensor((wl.B, wl.heads, wl.H, wl.W), torch.float32)
    rc = lib.rib_window_attn_fwd_gated(P(gpu["q"]), P(gpu["k"]), P(gpu["v"]), P(gpu["pq"]), P(gpu["pk"]), 0, P(gate), wl.B, wl.H, wl.W,
                                       wl.heads, wl.d, wl.r, wl.window, wl.shift, P(out), P(lse), None)
    assert rc == 0
    torch.cuda.synchronize()
    assert binding.rib_query_status() == 0
    g.check("gated forward")
    assert torch.equal(out, ref_out) and torch.equal(lse, ref_lse)


def test_cla_gate_and_generator_stay_inside_their_buffers():
    lib = binding.library()
    P = lambda t: t.data_ptr()
    B, H, W, D = 2, 16, 32, 192
    x = synthetic.bf16_tensor(67, "x", (B, H, W, D), 1.0).cuda()
    ws = [torch.randn(s, device="cuda") * 0.2 for s in ((D, 3, 3), (D,), (D, D), (D,))]
    ref = binding.rib_cla_gate(x, *ws)
    g = Guarded()
    gate = g.tensor((B, H, W, D), torch.bfloat16)
    assert lib.rib_cla_gate(P(x), *[P(w) for w in ws], B, H, W, D, P(gate), None) == 0
    torch.cuda.synchronize()
    assert binding.rib_query_status() == 0
    g.check("CLA gate")
    assert torch.equal(gate, ref)
    # backward of the gate: results and workspace guarded
    dgate = synthetic.bf16_tensor(68, "gate", (B, H, W, D), 1.0).cuda()
    ref = binding.rib_cla_gate_bwd(x, *ws, dgate)
    g = Guarded()
    dx = g.tensor((B, H, W, D), torch.bfloat16)
    grads = [g.tensor(tuple(w.shape), torch.float32) for w in ws]
    need = lib.rib_cla_gate_bwd_workspace(B, H, W, D)
    scratch = g.tensor((max(need, 256),), torch.uint8)
    rc = lib.rib_cla_gate_bwd(P(x), *[P(w) for w in ws], P(dgate), B, H, W, D, P(dx), *[P(t) for t in grads], P(scratch), scratch.numel(), None)
    assert rc == 0
    torch.cuda.synchronize()
    assert binding.rib_query_status() == 0
    g.check("CLA gate backward")
    assert torch.equal(dx, ref[0])
    for got, want in zip(grads, ref[1:]):
        torch.testing.assert_close(got, want, rtol=2e-3, atol=2e-3)     # fp32 atomic sums: order differs from run to run
    # feature generator (Eq. 1-3)
    window, L, dh, r = 16, 10, 32, 16
    gw = [torch.randn(s, device="cuda") * 0.3 for s in ((2 + 4 * L, dh), (dh,), (dh, r), (dh, r))]
    ref_pq, ref_pk = binding.rib_generate_features(*gw, window)
    g = Guarded()
    pq, pk = (g.tensor((window * window, r), torch.bfloat16) for _ in range(2))
    assert lib.rib_generate_features(*[P(w) for w in gw], window, L, dh, r, P(pq), P(pk), None) == 0
    torch.cuda.synchronize()
    g.check("feature generator")
    assert torch.equal(pq, ref_pq) and torch.equal(pk, ref_pk)


def test_a_repeated_call_encodes_no_tensor_map():
    wl = Workload("cache_w16_s8", 2, 32, 48, 2, 32, 16, 16, 8, seed=69)
    cpu, gpu = make(wl, with_dout=True)
    out, lse = run_fwd(gpu, wl)
    need = binding.rib_window_attn_bwd_workspace(wl.B, wl.H, wl.W, wl.heads, wl.d, wl.r, wl.window)
    ws = torch.empty(need, dtype=torch.uint8, device="cuda")
    call = lambda: (binding.rib_window_attn_fwd(gpu["q"], gpu["k"], gpu["v"], gpu["pq"], gpu["pk"], wl.window, wl.shift, out=out, lse=lse),
                    binding.rib_window_attn_bwd(gpu["q"], gpu["k"], gpu["v"], gpu["pq"], gpu["pk"], out, lse, gpu["dout"], wl.window, wl.shift,
                                                workspace=ws))
    call()
    hits0, misses0 = binding.rib_tensor_map_cache_counts()
    for _ in range(3):
        call()
    torch.cuda.synchronize()
    hits1, misses1 = binding.rib_tensor_map_cache_counts()
    assert misses1 == misses0 and hits1 == hits0 + 3 * 10      # 4 maps per forward, 6 per backward call
    assert binding.rib_query_status() == 0

"""Helpers shared by the GPU parity tests: run the CUDA path and the CPU oracle on the same
seeded bf16 inputs and compare element by element."""
from __future__ import annotations

import numpy as np
import torch

from oracle import rib_oracle as orc
from paper_2603_06738_b200 import binding, synthetic

# Tolerances of the parity contract: GPU (bf16 in, fp32 accumulate, bf16 out) against the fp64
# oracle on the same bf16-rounded inputs.
MAX_ABS = 1e-2
REL_L2 = 5e-3


def to_f64(t: torch.Tensor) -> np.ndarray:
    return t.detach().to("cpu", torch.float64).numpy()


def compare(name, got, ref, mask=None, max_abs=MAX_ABS, rel_l2=REL_L2):
    got, ref = np.asarray(got, dtype=np.float64), np.asarray(ref, dtype=np.float64)
    if mask is not None:
        got, ref = got[mask], ref[mask]
    assert got.shape == ref.shape and got.size > 0
    assert np.isfinite(got).all(), f"{name}: non-finite values in the GPU result"
    err = np.abs(got - ref).max()
    rl2 = np.linalg.norm(got - ref) / max(np.linalg.norm(ref), 1e-30)
    # shown with `pytest -s` / `-rP`: how much of each bound is used
    print(f"parity {name}: max|d|={err:.3e} (bound {max_abs:.1e}), rel-L2={rl2:.3e} (bound {rel_l2:.1e}), max|ref|={np.abs(ref).max():.3e}, n={got.size}")
    assert err <= max_abs and rl2 <= rel_l2, f"{name}: max|d|={err:.3e} (<= {max_abs}), rel-L2={rl2:.3e} (<= {rel_l2})"
    return err, rl2


def make(wl: synthetic.Workload, with_dout=True):
    cpu = synthetic.make_inputs(wl, with_dout=with_dout)
    gpu = {k: v.cuda() for k, v in cpu.items()}
    return cpu, gpu


def run_fwd(gpu, wl):
    fwd = binding.rib_window_attn_fwd_headwise if wl.headwise else binding.rib_window_attn_fwd
    out, lse = fwd(gpu["q"], gpu["k"], gpu["v"], gpu["pq"], gpu["pk"], wl.window, wl.shift)
    torch.cuda.synchronize()
    assert binding.rib_query_status() == 0
    return out, lse


def run_bwd(gpu, wl, out, lse):
    bwd = binding.rib_window_attn_bwd_headwise if wl.headwise else binding.rib_window_attn_bwd
    res = bwd(gpu["q"], gpu["k"], gpu["v"], gpu["pq"], gpu["pk"], out, lse, gpu["dout"], wl.window, wl.shift)
    torch.cuda.synchronize()
    assert binding.rib_query_status() == 0
    return res


def oracle_fwd(cpu, wl, pairs=None):
    return orc.fwd(*(to_f64(cpu[k]) for k in ("q", "k", "v", "pq", "pk")), wl.window, wl.shift, pairs=pairs)


def oracle_bwd(cpu, wl, pairs=None):
    return orc.bwd(*(to_f64(cpu[k]) for k in ("q", "k", "v", "pq", "pk", "dout")), wl.window, wl.shift, pairs=pairs)


def widths_fit_tensor_cores(d: int, r: int) -> bool:
    """Head width and rank that the tcgen05 kernels take: multiples of 8 up to 32 as they are, other even widths through
    zero-padded copies (a rank above 32 only when its columns above 32 fit the spare channels of the padded head)."""
    if d < 2 or d > 32 or r < 2 or d % 2 or r % 2:
        return False
    if d % 8 == 0 and r % 8 == 0:
        return r <= 32
    return r <= 32 or r - 32 <= (-d) % 8

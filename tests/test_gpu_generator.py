"""GPU parity of the RIB feature generator (Eq. 1-3) against its fp64 oracle, every element."""
import numpy as np
import pytest
import torch

from oracle import rib_generator_oracle as gen
from paper_2603_06738_b200 import binding

pytestmark = pytest.mark.gpu

# window, L, dh, r
CASES = [(1, 0, 4, 2), (4, 0, 8, 8), (6, 3, 16, 24), (16, 10, 32, 16), (32, 10, 32, 16), (48, 10, 32, 32), (20, 16, 64, 64)]


def _weights(L, dh, r, seed):
    rng = np.random.default_rng(seed)
    ws = (rng.normal(0, 0.3, (2 + 4 * L, dh)), rng.normal(0, 0.2, dh), rng.normal(0, 0.3, (dh, r)), rng.normal(0, 0.3, (dh, r)))
    return [np.float32(w) for w in ws]          # the GPU path takes fp32 weights; the oracle gets the same values


@pytest.mark.parametrize("window,L,dh,r", CASES)
def test_generator_forward_and_backward_match_the_oracle(window, L, dh, r):
    ws = _weights(L, dh, r, seed=window * 100 + L)
    gw = [torch.from_numpy(w).cuda() for w in ws]
    pq, pk = binding.rib_generate_features(*gw, window)
    ref_pq, ref_pk, _, _ = gen.forward(*ws, window, L)
    for name, got, ref in (("pq", pq, ref_pq), ("pk", pk, ref_pk)):
        got = got.double().cpu().numpy()
        scale = max(1.0, float(np.abs(ref).max()))
        assert np.abs(got - ref).max() <= 1e-2 * scale, name       # bf16 output: relative 2^-9 of values up to a few units
        assert np.linalg.norm(got - ref) <= 5e-3 * np.linalg.norm(ref), name
    rng = np.random.default_rng(7)
    dpq, dpk = np.float32(rng.normal(size=(window * window, r))), np.float32(rng.normal(size=(window * window, r)))
    got = binding.rib_generate_features_bwd(*gw, torch.from_numpy(dpq).cuda(), torch.from_numpy(dpk).cuda(), window)
    torch.cuda.synchronize()
    ref = gen.backward(*ws, dpq, dpk, window, L)
    for name, g, rf in zip(("dw_h", "db_h", "dw_pq", "dw_pk"), got, ref):
        g = g.double().cpu().numpy()
        scale = max(1.0, float(np.abs(rf).max()))
        assert np.abs(g - rf).max() <= 1e-3 * scale, name          # fp32 sums over at most 2304 tokens
        assert np.linalg.norm(g - rf) <= 1e-4 * max(np.linalg.norm(rf), 1e-30), name


def test_generated_features_feed_the_attention_entry_point():
    """Pq, Pk straight from the generator are valid pq / pk arguments of the attention forward."""
    window, L, dh, r = 16, 10, 32, 16
    gw = [torch.from_numpy(w).cuda() for w in _weights(L, dh, r, 3)]
    pq, pk = binding.rib_generate_features(*gw, window)
    q = torch.randn(1, 32, 32, 2, 32, device="cuda").to(torch.bfloat16)
    out, lse = binding.rib_window_attn_fwd(q, q, q, pq, pk, window, 8)
    torch.cuda.synchronize()
    assert binding.rib_query_status() == 0 and torch.isfinite(out.float()).all() and torch.isfinite(lse).all()


def test_generator_rejects_unsupported_sizes():
    lib = binding.library()
    args = [256, 512, 768, 1024]
    assert lib.rib_generate_features(*args, 16, 17, 32, 16, 2048, 4096, None) == -3
    assert lib.rib_generate_features(*args, 16, 10, 128, 16, 2048, 4096, None) == -3
    assert lib.rib_generate_features(*args, 0, 10, 32, 16, 2048, 4096, None) == -2
    assert lib.rib_generate_features(*args, 16, 10, 32, 16, None, 4096, None) == -1

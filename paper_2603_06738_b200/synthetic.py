"""Seeded synthetic inputs for RIB window attention.

This module only draws numbers: it holds none of the method's arithmetic, so both the CUDA
path and the CPU oracle may be fed from it.  The generator is counter based: element ``i`` of
tensor ``tensor_id`` under ``seed`` is a pure function of ``(seed, tensor_id, i)``, so a tensor
can be regenerated in any order or in slices.

Recipe (stands in for the query/key/value activations and RIB features of an SR transformer
layer, whose real statistics the paper does not give): q, k, v and the upstream gradient dout
are N(0, 1); the positional features pq, pk are N(0, 0.5^2); everything is rounded to bfloat16
with round-to-nearest-even and filled in memory order.
"""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np
import torch

TENSOR_IDS = {"q": 0, "k": 1, "v": 2, "pq": 3, "pk": 4, "dout": 5, "x": 6, "gate": 7}
_GOLDEN = np.uint64(0x9E3779B97F4A7C15)


def _splitmix64(z: np.ndarray) -> np.ndarray:
    """One round of the splitmix64 output function on an array of uint64 counters."""
    z = (z + _GOLDEN).astype(np.uint64)
    z = (z ^ (z >> np.uint64(30))) * np.uint64(0xBF58476D1CE4E5B9)
    z = (z ^ (z >> np.uint64(27))) * np.uint64(0x94D049BB133111EB)
    return z ^ (z >> np.uint64(31))


def normal(seed: int, tensor_id: int, count: int, sigma: float, start: int = 0) -> np.ndarray:
    """``count`` N(0, sigma^2) float64 samples, elements ``start .. start+count`` of the stream."""
    with np.errstate(over="ignore"):
        key = _splitmix64(np.array([np.uint64(seed) * np.uint64(0x100) + np.uint64(tensor_id)],
                                   dtype=np.uint64))[0]
        idx = np.arange(start, start + count, dtype=np.uint64)
        bits = _splitmix64(key + idx * _GOLDEN)
    u1 = ((bits >> np.uint64(32)).astype(np.float64) + 0.5) / 4294967296.0
    u2 = ((bits & np.uint64(0xFFFFFFFF)).astype(np.float64) + 0.5) / 4294967296.0
    return sigma * np.sqrt(-2.0 * np.log(u1)) * np.cos(2.0 * np.pi * u2)


def to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round float values to bfloat16 (nearest even); returns the 16-bit patterns as uint16."""
    u = np.asarray(x, dtype=np.float32).view(np.uint32)
    rounded = u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))
    return (rounded >> np.uint32(16)).astype(np.uint16)


def bf16_tensor(seed: int, name: str, shape, sigma: float) -> torch.Tensor:
    """A CPU torch.bfloat16 tensor of ``shape`` drawn from the stream of tensor ``name``."""
    count = int(np.prod(shape))
    bits = to_bf16_bits(normal(seed, TENSOR_IDS[name], count, sigma))
    return torch.from_numpy(bits.view(np.int16).reshape(shape)).view(torch.bfloat16)


@dataclass(frozen=True)
class Workload:
    """Shape of one problem: B images of H x W tokens, `heads` heads of width d, RIB rank r."""
    name: str
    B: int
    H: int
    W: int
    heads: int
    d: int
    r: int
    window: int
    shift: int
    seed: int
    backward: bool = False
    headwise: bool = False    # one Pq/Pk table per head ([heads, n, r]) instead of one for all heads

    @property
    def n(self) -> int:
        return self.window * self.window

    @property
    def tokens(self) -> int:
        return self.B * self.H * self.W

    @property
    def pairs(self) -> int:
        return self.B * (self.H // self.window) * (self.W // self.window) * self.heads

    @property
    def fwd_flops(self) -> int:
        return self.pairs * 2 * self.n * self.n * (2 * self.d + self.r)

    @property
    def bwd_flops(self) -> int:
        return self.pairs * 2 * self.n * self.n * (5 * self.d + 3 * self.r)


# The five benchmark configurations: shapes of SST-L / SST-L+ attention layers (6 heads of 32
# channels, rank 16, windows from the paper's window cycles, 96x96 training patches).
CONFIGS = (
    Workload("cfg1_fwd_b1_64x64_h2_w16_s0", 1, 64, 64, 2, 32, 16, 16, 0, seed=0),
    Workload("cfg2_fwd_b8_96x96_h6_w32_s16", 8, 96, 96, 6, 32, 16, 32, 16, seed=1),
    Workload("cfg3_fwd_b16_96x96_h6_w48_s24", 16, 96, 96, 6, 32, 16, 48, 24, seed=2),
    Workload("cfg4_fwd_b1_256x256_h6_w64_s32", 1, 256, 256, 6, 32, 16, 64, 32, seed=3),
    Workload("cfg5_fwdbwd_b16_96x96_h6_w32_s16", 16, 96, 96, 6, 32, 16, 32, 16, seed=4,
             backward=True),
)


def make_inputs(wl: Workload, with_dout: bool | None = None) -> dict[str, torch.Tensor]:
    """CPU bf16 tensors q, k, v [B,H,W,heads,d], pq, pk [n,r] or [heads,n,r] (and dout) for a workload."""
    shape = (wl.B, wl.H, wl.W, wl.heads, wl.d)
    t = {name: bf16_tensor(wl.seed, name, shape, 1.0) for name in ("q", "k", "v")}
    pos_shape = (wl.heads, wl.n, wl.r) if wl.headwise else (wl.n, wl.r)
    t["pq"] = bf16_tensor(wl.seed, "pq", pos_shape, 0.5)
    t["pk"] = bf16_tensor(wl.seed, "pk", pos_shape, 0.5)
    if wl.backward if with_dout is None else with_dout:
        t["dout"] = bf16_tensor(wl.seed, "dout", shape, 1.0)
    return t

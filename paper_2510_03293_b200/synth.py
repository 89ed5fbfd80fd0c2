"""Seeded synthetic routing workloads.

Input generation only: shapes, value distributions and parameter tables of the five
routing workloads.  Nothing in this module computes any part of the routing method, so
both the CUDA path's tests and the CPU checker may draw their inputs from it.

Recipe (per layer, stream id = 1000 * config index + layer or decode step):
  hidden[t,:] = bf16(s_t * z_t),  z_t ~ N(0, I_d),  s_t = exp(U[ln 0.1, ln 3])
  W_g[e,:]    = bf16(N(0, sigma^2))
  bias[e]     = (r_e^-alpha - E^-alpha) / (1 - E^-alpha), r a random permutation of 1..E
  expert_to_bin[e] = e // (E / B);  loads start at zero.
The per-token scale mixes flat (s = 0.1) and peaked (s = 3) softmax rows; the Zipf-ranked
bias makes some experts hot.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import List

import numpy as np


@dataclass(frozen=True)
class Workload:
    name: str
    index: int            # config index, used in the seed stream id
    layers: int           # independent MoE layers (or successive decode steps)
    T: int
    d: int
    E: int
    k: int
    c: int
    n_bins: int
    sigma: float
    alpha: float
    t_fix: float
    eps_high: tuple       # one value, or three (early / middle / final third of the layers)
    renormalize: int
    persistent_loads: bool = False   # decode stream: loads carried across steps

    def eps_for_layer(self, layer: int) -> float:
        if len(self.eps_high) == 1:
            return self.eps_high[0]
        third = min(2, (3 * layer) // max(1, self.layers))
        return self.eps_high[third]


# LASER parameters follow the paper's threshold table (Mixtral rows for E=8, DeepSeek rows
# for E=64) and the trimming sizes of its figures; the E=256 stress case has no paper value.
WORKLOADS = {
    "tiny":    Workload("tiny", 0, 1, 2048, 4096, 8, 2, 4, 4, 0.02, 1.2, 0.60, (0.6419,), 1),
    "mixtral": Workload("mixtral", 1, 32, 16384, 4096, 8, 2, 4, 8, 0.02, 1.2, 0.60,
                        (0.7159, 0.6419, 0.6285), 1),
    "deepseek": Workload("deepseek", 2, 27, 16384, 2048, 64, 6, 8, 8, 0.02, 1.1, 0.80, (0.40,), 0),
    "decode":  Workload("decode", 3, 4096, 64, 2048, 64, 6, 8, 8, 0.02, 1.1, 0.80, (0.40,), 0,
                        persistent_loads=True),
    "stress":  Workload("stress", 4, 1, 131072, 7168, 256, 8, 16, 32, 0.01, 1.3, 0.25, (0.30,), 1),
}


def f32_to_bf16_bits(a: np.ndarray) -> np.ndarray:
    """Round-to-nearest-even conversion of float32 values to bf16 bit patterns (uint16)."""
    u = np.ascontiguousarray(a, np.float32).view(np.uint32)
    rounded = u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))
    return (rounded >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(b, np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def _rng(seed: int, stream: int) -> np.random.Generator:
    return np.random.Generator(np.random.Philox(key=[seed, stream]))


def zipf_bias(E: int, alpha: float, rng: np.random.Generator) -> np.ndarray:
    ranks = rng.permutation(E).astype(np.float64) + 1.0
    if E == 1:
        return np.zeros((1,), np.float32)
    lo = float(E) ** (-alpha)
    return ((ranks ** (-alpha) - lo) / (1.0 - lo)).astype(np.float32)


def make_layer(T: int, d: int, E: int, sigma: float, alpha: float, seed: int = 0,
               stream: int = 0, with_bias: bool = True):
    """One layer's inputs as numpy arrays: hidden bits [T,d] u16, W_g bits [E,d] u16,
    bias [E] f32 (or None)."""
    rng = _rng(seed, stream)
    scale = np.exp(rng.uniform(np.log(0.1), np.log(3.0), size=(T, 1))).astype(np.float32)
    hidden = f32_to_bf16_bits(rng.standard_normal((T, d), dtype=np.float32) * scale)
    wg = f32_to_bf16_bits(rng.standard_normal((E, d), dtype=np.float32) * np.float32(sigma))
    bias = zipf_bias(E, alpha, rng) if with_bias else None
    return hidden, wg, bias


def make_workload_layer(w: Workload, layer: int, seed: int = 0, T: int | None = None):
    """Inputs of layer (or decode step) ``layer`` of a named workload; T may be reduced."""
    return make_layer(T if T is not None else w.T, w.d, w.E, w.sigma, w.alpha, seed,
                      1000 * w.index + layer)


def default_expert_to_bin(E: int, n_bins: int) -> np.ndarray:
    per = -(-E // n_bins)
    return (np.arange(E, dtype=np.int32) // per).astype(np.int32)


def make_workload_torch(w: Workload, device, seed: int = 0, layers: int | None = None):
    """All layers of a workload generated directly in device memory with torch's seeded
    generator (same recipe; a different random stream than the numpy path).

    Returns dict(hidden [L,T,d] bf16, w_g [L,E,d] bf16, bias [L,E] f32, eps_high list,
    t_fix list).
    """
    import torch

    L = layers if layers is not None else w.layers
    g = torch.Generator(device=device)
    g.manual_seed(seed * 1_000_003 + 1000 * w.index)
    hidden = torch.empty((L, w.T, w.d), dtype=torch.bfloat16, device=device)
    lo, hi = float(np.log(0.1)), float(np.log(3.0))
    for l in range(L):
        z = torch.randn((w.T, w.d), generator=g, device=device, dtype=torch.float32)
        s = torch.exp(torch.rand((w.T, 1), generator=g, device=device) * (hi - lo) + lo)
        hidden[l] = (z * s).to(torch.bfloat16)
        del z, s
    wg = (torch.randn((L, w.E, w.d), generator=g, device=device, dtype=torch.float32)
          * w.sigma).to(torch.bfloat16)
    bias = torch.empty((L, w.E), dtype=torch.float32, device=device)
    for l in range(L):
        b = zipf_bias(w.E, w.alpha, _rng(seed, 1000 * w.index + l))
        bias[l] = torch.from_numpy(b).to(device)
    return dict(hidden=hidden, w_g=wg, bias=bias,
                eps_high=[w.eps_for_layer(l) for l in range(L)],
                t_fix=[w.t_fix] * L)

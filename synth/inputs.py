"""Seeded synthetic inputs shared by the oracle-side tests and the CUDA-side tests/bench.

This module holds NO arithmetic of the method (no Hadamard transform, no grid
search, no scale, no sign function): only random draws with the shapes and
value distributions of the workloads, and exact dtype rounding helpers.  All
draws happen on the host with numpy so both sides see identical bits.

Recipe (stands in for the Llama checkpoints the paper measured, which are not
available offline):
  weights      W = 0.02 * N(0,1); a Bernoulli(1e-3) mask of entries is REPLACED
               by 0.1 * Student-t(nu=3); fp32, or rounded to bf16.
  activations  N(0,1), optionally multiplied by one LogNormal(0,1) factor per
               input channel (shared by all tokens), then rounded to bf16.
  grid samples N(0, I_p), 2^18 points by default.
"""
from __future__ import annotations

from typing import Dict, List, Tuple

import numpy as np

GROUP = 1024

# (name, N_out, K_in) of the distinct linear-layer shapes of one transformer block.
LAYER_SETS: Dict[str, List[Tuple[str, int, int]]] = {
    "ref512": [("ref", 512, 1024)],
    "llama-3.2-1b": [("q", 2048, 2048), ("k", 512, 2048), ("v", 512, 2048), ("o", 2048, 2048),
                     ("gate", 8192, 2048), ("up", 8192, 2048), ("down", 2048, 8192)],
    "llama-3.1-8b": [("q", 4096, 4096), ("k", 1024, 4096), ("v", 1024, 4096), ("o", 4096, 4096),
                     ("gate", 14336, 4096), ("up", 14336, 4096), ("down", 4096, 14336)],
    "llama-3.1-70b": [("q", 8192, 8192), ("k", 1024, 8192), ("v", 1024, 8192), ("o", 8192, 8192),
                      ("gate", 28672, 8192), ("up", 28672, 8192), ("down", 8192, 28672)],
}
CONFIG_OF_SET = {"ref512": 0, "llama-3.2-1b": 1, "llama-3.1-8b": 2, "llama-3.1-70b": 4}


def bf16_round(a: np.ndarray) -> np.ndarray:
    """Round fp32 values to the nearest bf16 (ties to even); result is fp32 holding bf16 values."""
    u = np.ascontiguousarray(a, dtype=np.float32).view(np.uint32).astype(np.uint64)
    u = (u + 0x7FFF + ((u >> 16) & 1)) >> 16
    return (u.astype(np.uint32) << 16).view(np.float32).reshape(np.shape(a))


def bf16_bits(a: np.ndarray) -> np.ndarray:
    """uint16 bit patterns of fp32 values that are already bf16-representable."""
    return (np.ascontiguousarray(a, dtype=np.float32).view(np.uint32) >> 16).astype(np.uint16).reshape(np.shape(a))


def weight_seed(config: int, layer_index: int) -> int:
    return 1000 * config + layer_index


def activation_seed(config: int, B: int) -> int:
    return 5000 + 100 * config + B


def rht_seed(config: int) -> int:
    return 0x48494747 + config


def grid_sample_seed(p: int, n: int) -> int:
    return 18 + 1000 * p + n


def make_weights(N: int, K: int, seed: int, bf16: bool) -> np.ndarray:
    """fp32 [N][K]; bf16-representable if bf16=True."""
    rng = np.random.default_rng(seed)
    W = (0.02 * rng.standard_normal((N, K))).astype(np.float32)
    mask = rng.random((N, K)) < 1e-3
    cnt = int(mask.sum())
    W[mask] = (0.1 * rng.standard_t(3, size=cnt)).astype(np.float32)
    return bf16_round(W) if bf16 else W


def make_activations(B: int, K: int, seed: int, lognormal_channels: bool = False) -> np.ndarray:
    """fp32 [B][K] holding bf16-representable values."""
    rng = np.random.default_rng(seed)
    x = rng.standard_normal((B, K))
    if lognormal_channels:
        x = x * np.exp(rng.standard_normal(K))[None, :]
    return bf16_round(x.astype(np.float32))


def gaussian_samples(p: int, seed: int, log2_count: int = 18) -> np.ndarray:
    """float64 [2^log2_count][p] from N(0, I_p)."""
    rng = np.random.default_rng(seed)
    return rng.standard_normal((1 << log2_count, p))


def bitwidth_assignment(seed: int, layers: List[Tuple[str, int, int]], blocks: int = 8,
                        target: float = 3.5, tol: float = 0.02, choices=(3, 4)) -> List[List[int]]:
    """Seeded per-matrix bit widths whose parameter-weighted mean is within tol of target.

    Returns assignment[block][layer_index]; redraws until the weighted mean fits.
    """
    rng = np.random.default_rng(seed)
    sizes = np.array([n * k for _, n, k in layers], dtype=np.float64)
    for _ in range(100000):
        a = rng.choice(choices, size=(blocks, len(layers)))
        mean = float((a * sizes[None, :]).sum() / (blocks * sizes.sum()))
        if abs(mean - target) <= tol:
            return a.tolist()
    raise RuntimeError("no assignment found")

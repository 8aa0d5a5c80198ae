"""Seeded synthetic inputs shared by the oracle-side tests and the CUDA-side
tests / benchmark.

This module holds no arithmetic of the mixers: it only draws i.i.d. N(0,1)
tensors with the shapes of the five workload configurations (token grids of
DINOv3-L / DepthAnythingV2-L at high resolution) and, for bf16 workloads, rounds
them to bf16 on the host so that both sides receive exactly the same values.
"""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np
import torch

SEED_BASE = 26_636_000


@dataclass(frozen=True)
class Workload:
    """One workload configuration: token grid, batch, heads and element type."""
    name: str
    cfg: int
    B: int
    H: int
    Hg: int
    Wg: int
    D: int
    dtype: str          # "f32" or "bf16"
    win: int = 16       # square window edge used by W
    n_layers: int = 1

    @property
    def N(self) -> int:
        return self.Hg * self.Wg

    @property
    def shape(self):
        return (self.B, self.H, self.N, self.D)

    @property
    def tokens(self) -> int:
        return self.B * self.N


HYBRID_SCHEDULE = "LWLWLF" * 4   # F at layers 5, 11, 17, 23 (0-indexed); W at other odd layers

WORKLOADS = {
    "tiny":     Workload("tiny", 1, 1, 6, 16, 16, 64, "f32", win=8),
    "dinov3_l": Workload("dinov3_l", 2, 8, 16, 64, 64, 64, "bf16"),
    "dinov3_w": Workload("dinov3_w", 3, 8, 16, 64, 64, 64, "bf16"),
    "dav2_l":   Workload("dav2_l", 4, 4, 16, 73, 73, 64, "bf16"),
    "hybrid24": Workload("hybrid24", 5, 1, 16, 128, 128, 64, "bf16", n_layers=24),
}


def seed_for(cfg: int, layer: int, tensor: int) -> int:
    """tensor: 0 = q, 1 = k, 2 = v, 3.. = auxiliary weights."""
    return SEED_BASE + 1000 * cfg + 10 * layer + tensor


def normal(shape, seed: int, dtype: str = "f32") -> torch.Tensor:
    """i.i.d. N(0,1) CPU tensor; ``bf16`` = fp32 draw rounded to nearest-even."""
    x = np.random.default_rng(seed).standard_normal(tuple(shape), dtype=np.float32)
    t = torch.from_numpy(x)
    if dtype == "bf16":
        return t.to(torch.bfloat16)
    if dtype == "f32":
        return t
    raise ValueError(dtype)


def qkv(w: Workload, layer: int = 0, shape=None):
    """Q, K, V of one layer of workload ``w`` (CPU tensors in w.dtype)."""
    shape = w.shape if shape is None else shape
    return tuple(normal(shape, seed_for(w.cfg, layer, t), w.dtype) for t in range(3))


def custom_qkv(B, H, N, D, dtype="f32", seed=0):
    """Q, K, V for ad-hoc shapes (shape sweeps and edge cases)."""
    return tuple(normal((B, H, N, D), SEED_BASE + 7 * seed + t, dtype) for t in range(3))


def dwc_weights(C: int, R: int, k: int, seed: int):
    """Generator weights of the squeeze dynamic convolution, fp32:
    W1 ~ N(0, 1/C) [R, C], W2 ~ N(0, 1/R) [C*k*k, R], b1 = 0, b2 = 0 except the
    centre tap of every channel = 0.1."""
    rng = np.random.default_rng(seed)
    W1 = (rng.standard_normal((R, C), dtype=np.float32) / np.sqrt(C)).astype(np.float32)
    W2 = (rng.standard_normal((C * k * k, R), dtype=np.float32) / np.sqrt(R)).astype(np.float32)
    b1 = np.zeros((R,), dtype=np.float32)
    b2 = np.zeros((C, k, k), dtype=np.float32)
    b2[:, k // 2, k // 2] = 0.1
    return {"k": k, "R": R, "W1": torch.from_numpy(W1), "b1": torch.from_numpy(b1),
            "W2": torch.from_numpy(W2), "b2": torch.from_numpy(b2.reshape(-1))}


def proj_weights(rows: int, C: int, seed: int, with_bias: bool = True):
    """Weights of a linear projection as a trained layer would hold them: w ~ N(0, 1/C)
    [rows, C] rounded to bf16, bias ~ 0.1 N(0, 1) fp32 [rows] (or None)."""
    rng = np.random.default_rng(seed)
    w = (rng.standard_normal((rows, C), dtype=np.float32) / np.sqrt(C)).astype(np.float32)
    b = (0.1 * rng.standard_normal((rows,), dtype=np.float32)).astype(np.float32) if with_bias else None
    return torch.from_numpy(w).to(torch.bfloat16), (None if b is None else torch.from_numpy(b))

"""The five synthetic workloads (shapes and statistics only; no benchmark item is reproduced).

Each stands in for document pages pushed through a Qwen2.5-VL-style decoder: N visual tokens on
a patch grid in raster order between a short system prefix and a text suffix, with a small,
slowly drifting fixation window receiving most of the image attention.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field
from typing import List

import numpy as np

BASE_SEED = 20260517


def kept_count_hint(n: int, tau: float) -> int:
    """ceil(tau*n) clamped to [0, n]; bookkeeping for buffer sizes only."""
    return max(0, min(n, math.ceil(tau * n - 1e-9)))


@dataclass
class WorkloadConfig:
    name: str
    seed: int
    layers: int
    num_q_heads: int
    num_kv_heads: int
    head_dim: int
    batch: int
    grid_h: List[int]            # per sequence
    grid_w: List[int]
    text_before: List[int]       # system/prompt tokens ahead of the image
    text_after: List[int]        # prompt tokens behind the image (at step 0)
    steps: int
    advance: int                 # fixation drift, patches per step
    tau: float
    rho: float = 0.1
    gap: int = 1
    warmup: int = 10
    page_size: int = 0           # 0 = contiguous
    notes: str = ""
    extra: dict = field(default_factory=dict)

    @property
    def vis_len(self):
        return [h * w for h, w in zip(self.grid_h, self.grid_w)]

    @property
    def vis_start(self):
        return list(self.text_before)

    def seq_len(self, step: int = 0):
        return [b + n + a + step for b, n, a in zip(self.text_before, self.vis_len, self.text_after)]


def get_config(name: str, **over) -> WorkloadConfig:
    n7 = dict(num_q_heads=28, num_kv_heads=4, head_dim=128)
    if name == "cfg0":      # single layer, single sequence, one step
        c = WorkloadConfig("cfg0", BASE_SEED + 0, 1, batch=1, grid_h=[32], grid_w=[32],
                           text_before=[16], text_after=[48], steps=1, advance=0, tau=0.05, **n7)
    elif name == "cfg1":    # 7B-shaped decode, one sequence
        c = WorkloadConfig("cfg1", BASE_SEED + 1, 28, batch=1, grid_h=[64], grid_w=[64],
                           text_before=[16], text_after=[240], steps=256, advance=4, tau=0.05, **n7)
    elif name == "cfg2":    # batched serving, ragged + paged
        rng = np.random.RandomState(BASE_SEED + 2)
        B = 32
        rows = rng.randint(64, 129, size=B)
        text = rng.randint(128, 513, size=B)
        c = WorkloadConfig("cfg2", BASE_SEED + 2, 28, batch=B, grid_h=[int(r) for r in rows],
                           grid_w=[64] * B, text_before=[16] * B,
                           text_after=[int(t) - 16 for t in text], steps=128, advance=4,
                           tau=0.05, page_size=16, **n7)
    elif name == "cfg3":    # 72B-shaped long page
        B = 8
        c = WorkloadConfig("cfg3", BASE_SEED + 3, 80, num_q_heads=64, num_kv_heads=8, head_dim=128,
                           batch=B, grid_h=[128] * B, grid_w=[128] * B, text_before=[16] * B,
                           text_after=[496] * B, steps=64, advance=8, tau=0.05)
    elif name == "cfg4":    # one point of the roofline sweep; N and tau overridable
        B = int(over.pop("batch", 64))
        N = int(over.pop("N", 8192))
        w = 1 << (int(math.log2(N)) // 2)
        h = N // w
        c = WorkloadConfig("cfg4", BASE_SEED + 4, int(over.pop("layers", 1)), batch=B,
                           grid_h=[h] * B, grid_w=[w] * B, text_before=[16] * B,
                           text_after=[240] * B, steps=int(over.pop("steps", 1)), advance=4,
                           tau=float(over.pop("tau", 0.05)), **n7)
    else:
        raise KeyError(name)
    for k, v in over.items():
        setattr(c, k, v)
    return c

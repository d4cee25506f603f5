"""Counter-based, device-independent input generator.

Every value is a pure function of (seed, stream, element index), computed with
integer tensor ops only, so the same bytes come out on CPU and on a CUDA device
and any slice of a large tensor can be regenerated without the rest.

Normal deviates: three 64-bit hash words per element are split into twelve
16-bit uniforms whose sum, centred and divided by 2**16, has unit variance
(the classical twelve-uniform approximation of N(0,1)); the result is exact in
fp32 and is rounded to bf16 (round-to-nearest-even) by the tensor cast.
"""
from __future__ import annotations

import math
from typing import Iterable, Sequence, Tuple

import numpy as np
import torch

_MASK64 = (1 << 64) - 1
_GOLD = 0x9E3779B97F4A7C15
_M1 = 0xBF58476D1CE4E5B9
_M2 = 0x94D049BB133111EB


def _s64(x: int) -> int:
    """Python int (mod 2**64) -> the signed value torch.int64 stores."""
    x &= _MASK64
    return x - (1 << 64) if x >= (1 << 63) else x


def _mix_py(z: int) -> int:
    z &= _MASK64
    z = ((z ^ (z >> 30)) * _M1) & _MASK64
    z = ((z ^ (z >> 27)) * _M2) & _MASK64
    return z ^ (z >> 31)


def stream_key(seed: int, *ids: int) -> int:
    """Fold a seed and a tuple of small integers (config, layer, tensor, ...) into a 64-bit key."""
    k = _mix_py(seed + _GOLD)
    for i in ids:
        k = _mix_py(k ^ ((int(i) + 1) * _GOLD))
    return k


def _lsr(z: torch.Tensor, s: int) -> torch.Tensor:
    return (z >> s) & ((1 << (64 - s)) - 1)


def _mix_t(z: torch.Tensor) -> torch.Tensor:
    z = (z ^ _lsr(z, 30)) * _s64(_M1)
    z = (z ^ _lsr(z, 27)) * _s64(_M2)
    return z ^ _lsr(z, 31)


def _normal_f32(key: int, start: int, count: int, device) -> torch.Tensor:
    idx = torch.arange(start, start + count, dtype=torch.int64, device=device)
    total = torch.zeros(count, dtype=torch.int64, device=device)
    for j in range(3):
        w = _mix_t(idx * 3 + j + _s64(key))
        total += (w & 0xFFFF) + (_lsr(w, 16) & 0xFFFF) + (_lsr(w, 32) & 0xFFFF) + _lsr(w, 48)
    return (total - 6 * 65535).to(torch.float32) / 65536.0


def normal_bf16(key: int, shape: Sequence[int], device="cpu", offset: int = 0,
                chunk: int = 1 << 24) -> torch.Tensor:
    """bf16 tensor of approximately N(0,1) values; element i (flat) depends only on (key, offset+i)."""
    n = int(math.prod(shape))
    out = torch.empty(n, dtype=torch.bfloat16, device=device)
    for s in range(0, n, chunk):
        c = min(chunk, n - s)
        out[s:s + c] = _normal_f32(key, offset + s, c, device).to(torch.bfloat16)
    return out.view(*shape)


def make_kv(seed: int, layer: int, batch: int, tokens: int, num_kv_heads: int, head_dim: int,
            device="cpu", seq_offset: int = 0, token_stride: int | None = None
            ) -> Tuple[torch.Tensor, torch.Tensor]:
    """K and V caches [batch][tokens][num_kv_heads][head_dim] (bf16) for one layer.

    Row j of sequence b is a function of (seed, layer, b + seq_offset, j) alone, so a cache
    grown by one token per step keeps its earlier rows and a single sequence can be rebuilt
    on another device. token_stride (>= tokens) fixes the per-sequence counter stride so that
    slices generated with different `tokens` agree.
    """
    stride = tokens if token_stride is None else token_stride
    row = num_kv_heads * head_dim
    outs = []
    for tensor_id in (0, 1):
        key = stream_key(seed, 101, layer, tensor_id)
        if stride == tokens:      # the whole tensor is one contiguous counter range
            t = normal_bf16(key, (batch, tokens, num_kv_heads, head_dim), device, offset=seq_offset * stride * row)
        else:
            t = torch.empty(batch, tokens, num_kv_heads, head_dim, dtype=torch.bfloat16, device=device)
            for b in range(batch):
                t[b] = normal_bf16(key, (tokens, num_kv_heads, head_dim), device,
                                   offset=(b + seq_offset) * stride * row)
        outs.append(t)
    return outs[0], outs[1]


def window_indices(centres: torch.Tensor, grid_h: torch.Tensor, grid_w: torch.Tensor):
    """Raster indices of the 3x3 patch window around each centre, with a validity mask.

    centres: int64 [B][2] (row, col); grid_h, grid_w: int64 [B]. Returns (idx [B][9], valid [B][9]).
    """
    dy = torch.tensor([-1, -1, -1, 0, 0, 0, 1, 1, 1], dtype=torch.int64, device=centres.device)
    dx = torch.tensor([-1, 0, 1, -1, 0, 1, -1, 0, 1], dtype=torch.int64, device=centres.device)
    r = centres[:, 0:1] + dy[None, :]
    c = centres[:, 1:2] + dx[None, :]
    valid = (r >= 0) & (r < grid_h[:, None]) & (c >= 0) & (c < grid_w[:, None])
    idx = torch.where(valid, r * grid_w[:, None] + c, torch.zeros_like(r))
    return idx, valid


def make_queries(seed: int, layer: int, step: int, k_rows, vis_start: torch.Tensor,
                 centres: torch.Tensor, grid_h: torch.Tensor, grid_w: torch.Tensor,
                 num_q_heads: int, seq_offset: int = 0) -> torch.Tensor:
    """Queries [B][H][d] (bf16): 2 x (mean key over the 3x3 fixation window) + N(0,1) noise per head.

    k_rows(b_idx, pos) -> bf16 [B][Hkv][d]: fetches one logical cache row per sequence (this keeps
    the function independent of contiguous vs paged storage). The window mean is accumulated in
    fp32 in a fixed order so CPU and GPU agree bit for bit.
    """
    device = centres.device
    B = centres.shape[0]
    idx, valid = window_indices(centres, grid_h, grid_w)
    b_idx = torch.arange(B, device=device)
    acc = None
    for w in range(9):
        rows = k_rows(b_idx, vis_start + idx[:, w]).to(torch.float32)
        rows = rows * valid[:, w].to(torch.float32)[:, None, None]
        acc = rows if acc is None else acc + rows
    count = valid.sum(dim=1).to(torch.float32)[:, None, None]
    mean2 = acc * 2.0 / count                                  # [B][Hkv][d]
    Hkv, d = mean2.shape[1], mean2.shape[2]
    G = num_q_heads // Hkv
    key = stream_key(seed, 202, layer, step)
    eps = torch.empty(B, num_q_heads, d, dtype=torch.bfloat16, device=device)
    for b in range(B):
        eps[b] = normal_bf16(key, (num_q_heads, d), device, offset=(b + seq_offset) * num_q_heads * d)
    q = mean2.repeat_interleave(G, dim=1) + eps.to(torch.float32)
    return q.to(torch.bfloat16)


def fixation_track(seed: int, seq: int, steps: int, grid_h: int, grid_w: int,
                   advance: int, jitter_sigma: float = 1.5) -> np.ndarray:
    """Fixation centres [steps][2] (row, col): a base point moving `advance` patches per step in
    raster order (wrapping from the last row to the first) plus independent Gaussian jitter per
    step (not accumulated), rounded and clamped to the grid."""
    rng = np.random.RandomState((stream_key(seed, 303, seq) & 0x7FFFFFFF))
    start = int(rng.randint(0, grid_h * grid_w))
    jit = rng.normal(0.0, jitter_sigma, size=(steps, 2))
    out = np.empty((steps, 2), dtype=np.int64)
    for t in range(steps):
        lin = (start + t * advance) % (grid_h * grid_w)
        r = int(np.clip(np.rint(lin // grid_w + jit[t, 0]), 0, grid_h - 1))
        c = int(np.clip(np.rint(lin % grid_w + jit[t, 1]), 0, grid_w - 1))
        out[t] = (r, c)
    return out


def make_page_table(seed: int, seq_tokens: Iterable[int], page_size: int, spare_pages: int = 0):
    """Shuffled physical page assignment. Returns (block_table int32 [B][max_pages] with -1 for
    unused slots, num_pages)."""
    need = [(int(s) + page_size - 1) // page_size for s in seq_tokens]
    total = sum(need) + spare_pages
    g = torch.Generator().manual_seed(stream_key(seed, 404) & 0x7FFFFFFF)
    perm = torch.randperm(total, generator=g).to(torch.int32)
    table = torch.full((len(need), max(need) if need else 0), -1, dtype=torch.int32)
    p = 0
    for b, n in enumerate(need):
        table[b, :n] = perm[p:p + n]
        p += n
    return table, total


def scatter_to_pages(logical: torch.Tensor, seq_tokens: Sequence[int], block_table: torch.Tensor,
                     num_pages: int, page_size: int, fill: float = 0.0) -> torch.Tensor:
    """Copy logical rows [B][S_max][Hkv][d] into a pool [num_pages][page_size][Hkv][d]."""
    B, _, Hkv, d = logical.shape
    pool = torch.full((num_pages, page_size, Hkv, d), fill, dtype=logical.dtype, device=logical.device)
    for b in range(B):
        S = int(seq_tokens[b])
        n = (S + page_size - 1) // page_size
        pages = block_table[b, :n].to(torch.int64).to(logical.device)
        padded = torch.full((n * page_size, Hkv, d), fill, dtype=logical.dtype, device=logical.device)
        padded[:S] = logical[b, :S]
        pool[pages] = padded.view(n, page_size, Hkv, d)
    return pool

"""Shared test scaffolding: builds one seeded batch both as oracle inputs (per-sequence CPU tensors)
and as device buffers for the CUDA library. Pure data movement; no attention arithmetic here."""
from __future__ import annotations

import math
from dataclasses import dataclass
from typing import List, Optional

import torch

from workloads import make_kv, make_queries, make_page_table, scatter_to_pages

SCALE = 1.0 / math.sqrt(128.0)


@dataclass
class Case:
    B: int
    H: int
    Hkv: int
    seq_len: List[int]
    vis_start: List[int]
    vis_len: List[int]
    K: torch.Tensor            # CPU bf16 [B][Smax][Hkv][128] logical
    V: torch.Tensor
    q: torch.Tensor            # CPU bf16 [B][H][128]
    page_size: int = 0
    block_table: Optional[torch.Tensor] = None
    num_pages: int = 0

    def seq(self, b):
        S = self.seq_len[b]
        return self.q[b], self.K[b, :S].contiguous(), self.V[b, :S].contiguous()

    def device_view(self, dev="cuda", poison=False, extra_stride=0):
        from paper_2605_17447_b200 import KVView
        i32 = lambda x: torch.tensor(x, dtype=torch.int32, device=dev)
        if self.page_size:
            fill = float("nan") if poison else 0.0
            kp = scatter_to_pages(self.K, self.seq_len, self.block_table, self.num_pages, self.page_size, fill)
            vp = scatter_to_pages(self.V, self.seq_len, self.block_table, self.num_pages, self.page_size, fill)
            bt = self.block_table.clone()
            bt[bt < 0] = 0
            return KVView(kp.to(dev), vp.to(dev), i32(self.seq_len), i32(self.vis_start), i32(self.vis_len), self.H,
                          max(self.seq_len), SCALE, block_table=bt.to(dev))
        K, V = self.K, self.V
        if poison or extra_stride:
            Smax = K.shape[1] + extra_stride
            K2 = torch.full((self.B, Smax, self.Hkv, 128), float("nan") if poison else 0.0, dtype=torch.bfloat16)
            V2 = K2.clone()
            for b in range(self.B):
                K2[b, :self.seq_len[b]] = K[b, :self.seq_len[b]]
                V2[b, :self.seq_len[b]] = V[b, :self.seq_len[b]]
            K, V = K2, V2
        return KVView(K.to(dev), V.to(dev), i32(self.seq_len), i32(self.vis_start), i32(self.vis_len), self.H,
                      max(self.seq_len), SCALE)


def make_case(seed, spans, H=28, Hkv=4, page_size=0, grid_w=None, boost=2.0) -> Case:
    """spans: list of (text_before, n_vis, text_after) per sequence."""
    B = len(spans)
    seq_len = [a + n + c for a, n, c in spans]
    vis_start = [a for a, _, _ in spans]
    vis_len = [n for _, n, _ in spans]
    Smax = max(seq_len)
    K, V = make_kv(seed, 0, B, Smax, Hkv, 128)
    gw = [grid_w or max(1, int(math.isqrt(max(n, 1)))) for n in vis_len]
    gh = [max(1, n // w) for n, w in zip(vis_len, gw)]
    g = torch.Generator().manual_seed(seed)
    centres = torch.stack([torch.tensor([int(torch.randint(0, h, (1,), generator=g)), int(torch.randint(0, w, (1,), generator=g))])
                           for h, w in zip(gh, gw)])
    has_vis = all(n > 0 for n in vis_len)
    if has_vis:
        q = make_queries(seed, 0, 0, lambda b, pos: K[b, pos], torch.tensor(vis_start), centres,
                         torch.tensor(gh), torch.tensor(gw), H)
    else:
        from workloads import normal_bf16, stream_key
        q = normal_bf16(stream_key(seed, 5), (B, H, 128))
    case = Case(B, H, Hkv, seq_len, vis_start, vis_len, K, V, q, page_size)
    if page_size:
        case.block_table, case.num_pages = make_page_table(seed, seq_len, page_size, spare_pages=3)
    return case


def make_layer_stack(seed, spans, L, H=28, Hkv=4, page_size=0, q_boost=1.0):
    """L layers over one batch geometry: per-layer K, V and queries (all seeded), the views sharing one
    set of length arrays as a caller's would. -> (cases per layer, views per layer, q [L][B][H][128] CPU)."""
    from paper_2605_17447_b200 import KVView
    from workloads import normal_bf16, stream_key
    base = make_case(seed, spans, H=H, Hkv=Hkv, page_size=page_size)
    cases, views, shared = [], [], None
    for l in range(L):
        K, V = make_kv(seed, l, base.B, max(base.seq_len), Hkv, 128)
        q = normal_bf16(stream_key(seed, 55, l), (base.B, H, 128))
        if q_boost != 1.0:
            q = (q.float() * q_boost).to(torch.bfloat16)
        c = Case(base.B, H, Hkv, base.seq_len, base.vis_start, base.vis_len, K, V, q, base.page_size,
                 base.block_table, base.num_pages)
        cases.append(c)
        v = c.device_view()
        if shared is None:
            shared = (v.seq_len, v.vis_start, v.vis_len)
        views.append(KVView(v.k, v.v, shared[0], shared[1], shared[2], H, max(base.seq_len), SCALE,
                            block_table=v.block_table if page_size else None))
    return cases, views, torch.stack([c.q for c in cases])

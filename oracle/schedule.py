"""Algorithm 1 written over the oracle primitives (test infrastructure only).

One sequence at a time. `layers` is a list of (q [H][d], K [S][Hkv][d], V [S][Hkv][d]) bf16
CPU tensors, one triple per transformer layer, for the current decode step.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import List, Optional, Sequence

import torch

from . import binding as ob


@dataclass
class StepTrace:
    outputs: List[torch.Tensor] = field(default_factory=list)      # per layer, [H][d] fp32
    mode: List[str] = field(default_factory=list)                  # "focal" | "pruned"
    used_set: List[Optional[torch.Tensor]] = field(default_factory=list)  # idx the layer attended (None = full)
    selected: List[Optional[torch.Tensor]] = field(default_factory=list)  # idx the layer produced (focal only)
    f_last: Optional[torch.Tensor] = None                          # state after the step


def _union(a: torch.Tensor, b: torch.Tensor) -> torch.Tensor:
    """Set union of two index lists, ascending."""
    return torch.tensor(sorted(set(a.tolist()) | set(b.tolist())), dtype=torch.int32)


def decode_step(layers, focal: Sequence[int], f_last: Optional[torch.Tensor], vis_start: int, N: int,
                tau: float, sm_scale: float, acc64: bool = False, union_sets: bool = False) -> StepTrace:
    """One post-warm-up decode step (Algorithm 1, the Cross-Step Fixation Reuse and Cross-Layer
    Propagation blocks).

    Layer 0 borrows last step's set when it is not focal and a set exists; otherwise it attends
    the full cache and selects (the fallback). Every later focal layer attends the full cache and
    refreshes the set; every other layer attends text + current set. The set left by the deepest
    focal layer (or by the fallback when no layer is focal) is kept for the next step.

    union_sets (a variant; Section 3.1.1 speaks of the aggregated set, the union over the focal
    layers of F^t_{l_i}): the kept image set after a focal layer is the union of the sets selected
    so far in THIS step (the first selection of a step replaces what was borrowed from the previous
    step, later ones are added); what is carried to the next step stays the deepest focal layer's
    own selection, as in Algorithm 1.
    """
    C = set(int(c) for c in focal)
    k = ob.kept_count(N, tau)
    tr = StepTrace()
    current: Optional[torch.Tensor] = None
    deepest: Optional[torch.Tensor] = None
    step_union: Optional[torch.Tensor] = None          # union of this step's selections (union_sets only)
    for li, (q, K, V) in enumerate(layers):
        is_focal = li in C
        if li == 0 and not is_focal and f_last is not None:
            current = f_last
        if is_focal or (li == 0 and current is None):
            out = ob.dense(q, K, V, sm_scale, acc64)
            sc, _ = ob.scores(q, K, sm_scale, vis_start, N, acc64)
            chosen = ob.topk(sc, k)
            if is_focal or not C:
                deepest = chosen
            current = _union(step_union, chosen) if (union_sets and step_union is not None) else chosen
            step_union = current
            tr.mode.append("focal")
            tr.used_set.append(None)
            tr.selected.append(chosen)
        else:
            out = ob.sparse(q, K, V, sm_scale, vis_start, N, current, acc64)
            tr.mode.append("pruned")
            tr.used_set.append(current)
            tr.selected.append(None)
        tr.outputs.append(out)
    tr.f_last = deepest if deepest is not None else f_last
    return tr


def warmup_step(layers, vis_start: int, N: int, sm_scale: float, acc64: bool = False):
    """One warm-up step (Algorithm 1, profiling block; Section 3.1.1): every layer attends the full
    cache, nothing is pruned, and Eq. 1's image-attention ratio r_i is recorded per layer.
    -> (outputs per layer [H][d], ratios per layer)."""
    outs, ratios = [], []
    for q, K, V in layers:
        outs.append(ob.dense(q, K, V, sm_scale, acc64))
        ratios.append(ob.scores(q, K, sm_scale, vis_start, N, acc64)[1])
    return outs, ratios


def profile_focal_layers(ratios_per_step, rho: float, gap: int):
    """Focal Layer Selection from warm-up records: ratios_per_step[t][l] = Eq. 1's r for layer l at
    warm-up step t. Mean over the w steps, then rank + greedy gap rule."""
    w = len(ratios_per_step)
    L = len(ratios_per_step[0])
    mean = [sum(float(ratios_per_step[t][l]) for t in range(w)) / w for l in range(L)]
    return ob.focal_layers(mean, rho, gap)

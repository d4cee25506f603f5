"""Pins for the oracle's integer rules, cost formula and Algorithm-1 schedule (no GPU)."""
import json
import math
import os

import torch

import oracle
from workloads import normal_bf16, stream_key, make_kv

GOLD = json.load(open(os.path.join(os.path.dirname(__file__), "golden", "paper_values.json")))
SCALE = 1.0 / math.sqrt(128.0)


def test_attention_flops_reproduce_printed_values():
    for row in GOLD["attn_flops_G"]:
        got = oracle.attn_flops(row["b"], row["l"], row["h"], row["s"]) / 1e9
        assert abs(got - row["printed"]) < 0.006, row["cite"]


def test_pruned_flops_reproduce_printed_values():
    for row in GOLD["attn_flops_pruned_G"]["rows"]:
        got = oracle.attn_flops_pruned(row["b"], row["l"], row["h"], row["s"], row["full_layers"], row["tau"] * row["s"]) / 1e9
        assert abs(got - row["printed"]) < row["tol"], (row["cite"], got)
    # special cases: every layer full = the vanilla count; no layer full, nothing kept = projections only
    assert oracle.attn_flops_pruned(8, 36, 2048, 4096, 36, 0) == oracle.attn_flops(8, 36, 2048, 4096)
    assert oracle.attn_flops_pruned(2, 10, 64, 999, 0, 0) == 2 * 10 * 8 * 64 * 64
    # a dropped projection term on the pruned layers, or tau*s swapped for s, would miss the printed values by > 1 G
    assert abs(oracle.attn_flops_pruned(8, 36, 2048, 4096, 4, 4096) / 1e9 - 19.33) < 0.006


def test_kept_count_is_a_ceiling():
    assert oracle.kept_count(1024, 0.05) == 52          # 51.2 -> 52 (a floor would give 51)
    assert [oracle.kept_count(n, 0.05) for n in (4096, 8192, 16384, 32768)] == [205, 410, 820, 1639]
    assert oracle.kept_count(4096, 0.25) == 1024        # exact product stays exact
    assert oracle.kept_count(1000, 0.004) == 4 and oracle.kept_count(4096, 0.004) == 17
    assert oracle.kept_count(77, 0.0) == 0 and oracle.kept_count(77, 1.0) == 77 and oracle.kept_count(77, 2.0) == 77
    assert oracle.kept_count(20, 0.05) == 1 and oracle.kept_count(100, 0.1) == 10


def test_focal_budget_matches_printed_counts():
    for row in GOLD["focal_layer_budget"]:
        ratios = [1.0 / (3 + 7 * ((l * 37) % row["L"])) for l in range(row["L"])]   # distinct, scattered
        assert len(oracle.focal_layers(ratios, row["rho"], 0)) == row["count"], row["cite"]
    assert len(oracle.focal_layers([0.1 * i for i in range(28)], 0.1, 0)) == 2
    assert len(oracle.focal_layers([0.1 * i for i in range(80)], 0.1, 0)) == 8
    assert oracle.focal_layers([0.5] * 5, 0.1, 1) == []  # floor(0.5) = 0: no focal layer at all


def test_focal_gap_rule_is_strict():
    g = GOLD["focal_gap"]
    L = 34
    ratios = [0.01] * L
    for rank, l in enumerate(g["always_focal"]):
        ratios[l] = 0.9 - 0.01 * rank
    # layers two apart are all accepted at g=1 ...
    assert oracle.focal_layers(ratios, 0.2, g["g"])[:5] == g["always_focal"] or \
        set(g["always_focal"]) <= set(oracle.focal_layers(ratios, 0.2, g["g"]))
    # ... while a neighbour of an accepted layer is skipped even when it ranks second
    ratios2 = [0.0] * 10
    ratios2[4], ratios2[5], ratios2[7], ratios2[1] = 0.9, 0.8, 0.7, 0.6
    assert oracle.focal_layers(ratios2, 0.3, 1) == [1, 4, 7]
    assert oracle.focal_layers(ratios2, 0.3, 0) == [4, 5, 7]
    assert oracle.focal_layers(ratios2, 0.3, 2) == [1, 4, 7]
    # g=3: layers 1 and 7 are exactly 3 away from layer 4 and are skipped; the walk continues
    # down the ranking (zero-ratio layers, lower index first) until the budget of 3 is filled
    assert oracle.focal_layers(ratios2, 0.3, 3) == [0, 4, 8]
    # the gap can leave C below its budget
    assert oracle.focal_layers([0.9, 0.8, 0.7], 1.0, 5) == [0]


def test_profile_means_over_warmup_steps():
    steps = [[0.1, 0.9, 0.2, 0.3], [0.1, 0.1, 0.2, 0.9], [0.1, 0.2, 0.2, 0.9]]
    assert oracle.profile_focal_layers(steps, 0.5, 1) == [1, 3]


def _layers(seed, L, S, H=4, Hkv=2):
    out = []
    for l in range(L):
        K, V = make_kv(seed, l, 1, S, Hkv, 128)
        out.append((normal_bf16(stream_key(seed, 77, l), (H, 128)), K[0], V[0]))
    return out


def test_schedule_single_focal_layer_trace():
    # L=4, C={2}: step 1 has no previous set -> layer 0 falls back (dense + select), layer 1
    # inherits it, layer 2 refreshes, layer 3 inherits the refreshed set, which is kept.
    vs, N, tau = 4, 40, 0.1
    lay = _layers(1, 4, 50)
    t1 = oracle.decode_step(lay, [2], None, vs, N, tau, SCALE)
    assert t1.mode == ["focal", "pruned", "focal", "pruned"]
    assert torch.equal(t1.used_set[1], t1.selected[0]) and torch.equal(t1.used_set[3], t1.selected[2])
    assert torch.equal(t1.f_last, t1.selected[2]) and len(t1.f_last) == 4
    sc, _ = oracle.scores(lay[2][0], lay[2][1], SCALE, vs, N)
    assert torch.equal(t1.selected[2], oracle.topk(sc, 4))
    assert torch.equal(t1.outputs[2], oracle.dense(*lay[2], SCALE))
    assert torch.equal(t1.outputs[3], oracle.sparse(*lay[3], SCALE, vs, N, t1.selected[2]))
    # step 2: layers 0 and 1 reuse last step's set, no fallback
    lay2 = _layers(2, 4, 51)
    t2 = oracle.decode_step(lay2, [2], t1.f_last, vs, N, tau, SCALE)
    assert t2.mode == ["pruned", "pruned", "focal", "pruned"]
    assert torch.equal(t2.used_set[0], t1.f_last) and torch.equal(t2.used_set[1], t1.f_last)
    assert torch.equal(t2.f_last, t2.selected[2])


def test_schedule_layer0_focal_and_no_focal_layers():
    vs, N, tau = 3, 30, 0.2
    lay = _layers(3, 3, 40)
    prev = torch.arange(6, dtype=torch.int32)
    t = oracle.decode_step(lay, [0, 2], prev, vs, N, tau, SCALE)        # layer 0 focal: never reuses
    assert t.mode == ["focal", "pruned", "focal"] and torch.equal(t.used_set[1], t.selected[0])
    assert torch.equal(t.f_last, t.selected[2])
    t = oracle.decode_step(lay, [], None, vs, N, tau, SCALE)            # C empty: fallback feeds all layers
    assert t.mode == ["focal", "pruned", "pruned"] and torch.equal(t.f_last, t.selected[0])
    t = oracle.decode_step(lay, [], prev, vs, N, tau, SCALE)            # C empty with a set: pure reuse
    assert t.mode == ["pruned"] * 3 and torch.equal(t.f_last, prev)


def test_schedule_union_of_the_steps_selections():
    # L=5, C={1,3}: layer 0 borrows last step's set; layer 1 selects F1 (replaces the borrowed set);
    # layer 2 attends T u F1; layer 3 selects F3; layer 4 attends T u (F1 u F3) in the union variant
    # and T u F3 in Algorithm 1 itself; in both, F3 alone is carried to the next step.
    vs, N, tau = 5, 60, 0.1
    lay = _layers(7, 5, 70)
    prev = torch.tensor([0, 1, 2, 3, 4, 59], dtype=torch.int32)
    plain = oracle.decode_step(lay, [1, 3], prev, vs, N, tau, SCALE)
    uni = oracle.decode_step(lay, [1, 3], prev, vs, N, tau, SCALE, union_sets=True)
    assert uni.mode == plain.mode == ["pruned", "focal", "pruned", "focal", "pruned"]
    f1, f3 = plain.selected[1], plain.selected[3]
    assert torch.equal(uni.selected[1], f1) and torch.equal(uni.selected[3], f3)      # selections do not depend on the variant
    assert torch.equal(uni.used_set[0], prev) and torch.equal(uni.used_set[2], f1)
    both = sorted(set(f1.tolist()) | set(f3.tolist()))
    assert uni.used_set[4].tolist() == both and len(both) > len(f3)                    # the sets differ on this input
    assert torch.equal(plain.used_set[4], f3)
    assert torch.equal(uni.outputs[4], oracle.sparse(*lay[4], SCALE, vs, N, torch.tensor(both, dtype=torch.int32)))
    assert not torch.equal(uni.outputs[4], plain.outputs[4])
    for l in range(4):
        assert torch.equal(uni.outputs[l], plain.outputs[l])
    assert torch.equal(uni.f_last, f3) and torch.equal(plain.f_last, f3)
    # the fallback's selection at layer 0 counts as the step's first
    u2 = oracle.decode_step(lay, [3], None, vs, N, tau, SCALE, union_sets=True)
    assert u2.used_set[4].tolist() == sorted(set(u2.selected[0].tolist()) | set(u2.selected[3].tolist()))


def test_warmup_step_is_dense_everywhere_and_records_eq1():
    vs, N = 4, 40
    lay = _layers(9, 3, 50)
    outs, ratios = oracle.warmup_step(lay, vs, N, SCALE)
    for l in range(3):
        assert torch.equal(outs[l], oracle.dense(*lay[l], SCALE))
        p = oracle.probs(lay[l][0], lay[l][1], SCALE, True).double().mean(dim=0)     # head-averaged weights over the cache
        img, txt = p[vs:vs + N].sum(), p[:vs].sum() + p[vs + N:].sum()
        assert abs(ratios[l] - float(img / (img + txt))) < 1e-6 and 0 < ratios[l] < 1   # Eq. 1 written out

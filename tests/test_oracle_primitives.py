"""Pins for the CPU oracle's attention primitives (no GPU): library routines, closed forms and
identities that a dropped term, a wrong sign/index or a transposed operand would break."""
import math

import pytest
import torch

import oracle
from workloads import normal_bf16, stream_key, make_kv

SCALE = 1.0 / math.sqrt(128.0)


def _case(seed, S, H=28, Hkv=4, d=128):
    K, V = make_kv(seed, 0, 1, S, Hkv, d)
    q = normal_bf16(stream_key(seed, 9), (H, d))
    return q, K[0], V[0]


def _torch_attention(q, K, V, scale, keep=None):
    """softmax(q K^T * scale) V with library routines in fp64; GQA by repeating KV heads."""
    H, d = q.shape
    S, Hkv, _ = K.shape
    G = H // Hkv
    Kh = K.double().permute(1, 0, 2).repeat_interleave(G, dim=0)      # [H][S][d]
    Vh = V.double().permute(1, 0, 2).repeat_interleave(G, dim=0)
    logits = torch.einsum("hd,hsd->hs", q.double(), Kh) * scale
    if keep is not None:
        logits = logits.masked_fill(~keep[None, :], float("-inf"))
    p = torch.softmax(logits, dim=-1)
    return torch.einsum("hs,hsd->hd", p, Vh), p


@pytest.mark.parametrize("acc64", [False, True])
@pytest.mark.parametrize("S,H,Hkv", [(1, 28, 4), (37, 28, 4), (300, 64, 8), (129, 4, 2), (64, 3, 3)])
def test_dense_matches_library_softmax(S, H, Hkv, acc64):
    q, K, V = _case(11 + S, S, H, Hkv)
    ref, pref = _torch_attention(q, K, V, SCALE)
    out = oracle.dense(q, K, V, SCALE, acc64)
    p = oracle.probs(q, K, SCALE, acc64)
    tol = 1e-6 if acc64 else 2e-5
    assert (out.double() - ref).abs().max() < tol
    assert (p.double() - pref).abs().max() < tol
    assert (p.double().sum(dim=1) - 1).abs().max() < 1e-5


def test_gqa_mapping_is_contiguous_groups():
    # Make KV head 1 the only one whose values are non-zero: exactly heads G..2G-1 must see them.
    q, K, V = _case(5, 20, H=6, Hkv=3)
    V = V.clone()
    V[:, 0] = 0
    V[:, 2] = 0
    out = oracle.dense(q, K, V, SCALE)
    assert out[0:2].abs().max() == 0 and out[4:6].abs().max() == 0 and out[2:4].abs().min() > 0


def test_one_token_cache_returns_value_row_exactly():
    q, K, V = _case(3, 1)
    out = oracle.dense(q, K, V, SCALE)
    assert torch.equal(out, V[0].float().repeat_interleave(7, dim=0))


def test_constant_keys_give_mean_of_values():
    q, K, V = _case(4, 50)
    K = K[:1].expand(50, -1, -1).contiguous()
    out = oracle.dense(q, K, V, SCALE, acc64=True)
    mean = V.double().mean(dim=0).repeat_interleave(7, dim=0)
    assert (out.double() - mean).abs().max() < 1e-6


def test_scale_enters_the_logits():
    q, K, V = _case(6, 40)
    a = oracle.dense(q, K, V, SCALE, True)
    ref, _ = _torch_attention(q, K, V, 0.5 * SCALE)
    b = oracle.dense(q, K, V, 0.5 * SCALE, True)
    assert (b.double() - ref).abs().max() < 1e-6 and (a - b).abs().max() > 1e-3


@pytest.mark.parametrize("acc64", [False, True])
def test_scores_are_head_mean_of_full_softmax(acc64):
    q, K, V = _case(21, 200)
    vis_start, N = 16, 150
    _, p = _torch_attention(q, K, V, SCALE)
    ref = p.mean(dim=0)[vis_start:vis_start + N]
    sc, mass = oracle.scores(q, K, SCALE, vis_start, N, acc64)
    assert (sc.double() - ref).abs().max() < (1e-7 if acc64 else 2e-6)
    # Eq. 1: image mass + text mass = 1, so r = sum of the scores and 0 < r < 1
    text = p.mean(dim=0)[:vis_start].sum() + p.mean(dim=0)[vis_start + N:].sum()
    assert abs(mass + float(text) - 1.0) < 1e-5 and 0.0 < mass < 1.0
    assert abs(mass - float(sc.double().sum())) < 1e-6


def test_scores_softmax_is_over_full_cache_not_image_only():
    # Adding a dominant text token must shrink every image score (it would not if the softmax
    # were renormalised over the image span).
    q, K, V = _case(22, 80, H=4, Hkv=1)
    sc0, _ = oracle.scores(q, K, SCALE, 8, 64, True)
    K2 = K.clone()
    K2[2, 0] = (q[0].float() * 4).to(torch.bfloat16)
    sc1, _ = oracle.scores(q, K2, SCALE, 8, 64, True)
    assert sc1.sum() < 0.9 * sc0.sum()


def test_single_head_ranking_equals_logit_ranking():
    q, K, V = _case(23, 120, H=1, Hkv=1)
    sc, _ = oracle.scores(q, K, SCALE, 10, 100, True)
    logits = (K[10:110, 0].double() @ q[0].double())
    assert torch.equal(torch.argsort(sc.double(), descending=True, stable=True)[:20],
                       torch.argsort(logits, descending=True, stable=True)[:20])


def test_scores_permute_with_visual_tokens():
    q, K, V = _case(24, 90)
    perm = torch.randperm(64, generator=torch.Generator().manual_seed(1))
    K2 = K.clone()
    K2[10:74] = K[10:74][perm]
    a, _ = oracle.scores(q, K, SCALE, 10, 64, True)
    b, _ = oracle.scores(q, K2, SCALE, 10, 64, True)
    assert (a[perm] - b).abs().max() < 1e-7


# ---------------------------------------------------------------- top-k
def _rank_count_topk(s, k):
    """Brute force: token i is kept iff fewer than k tokens beat it (larger score, or an equal
    score at a lower index). NaN loses to everything."""
    n = len(s)
    key = [(-math.inf if math.isnan(x) else x) for x in s]
    nan = [math.isnan(x) for x in s]
    keep = []
    for i in range(n):
        beat = 0
        for j in range(n):
            if j == i:
                continue
            if nan[i] and not nan[j]:
                beat += 1
            elif nan[i] == nan[j] and (key[j] > key[i] or (key[j] == key[i] and j < i)):
                beat += 1
        if beat < k:
            keep.append(i)
    return keep


@pytest.mark.parametrize("seed", range(6))
def test_topk_matches_rank_counting_with_heavy_ties(seed):
    g = torch.Generator().manual_seed(seed)
    n = int(torch.randint(1, 65, (1,), generator=g))
    s = torch.randint(0, 4, (n,), generator=g).float() / 4            # many exact ties
    for k in sorted({0, 1, n // 3, n - 1 if n > 1 else 0, n}):
        assert oracle.topk(s, k).tolist() == _rank_count_topk(s.tolist(), k)


def test_topk_special_values():
    s = torch.tensor([0.0, -0.0, float("nan"), 1.0, float("-inf"), 1.0, float("inf"), -2.0])
    for k in range(len(s) + 1):
        assert oracle.topk(s, k).tolist() == _rank_count_topk(s.tolist(), k)
    assert oracle.topk(s, 3).tolist() == [3, 5, 6]          # inf, then the two 1.0
    assert oracle.topk(s, 5).tolist() == [0, 1, 3, 5, 6]    # +0 and -0 tie: both before -2
    assert oracle.topk(torch.full((9,), 0.25), 4).tolist() == [0, 1, 2, 3]


def test_topk_agrees_with_library_on_tie_free_input():
    s = torch.randperm(5000, generator=torch.Generator().manual_seed(3)).float() / 5000.0
    assert len(set(s.tolist())) == 5000
    for k in (1, 52, 250, 4999):
        assert oracle.topk(s, k).tolist() == torch.topk(s, k).indices.sort().values.tolist()


def test_topk_rejects_bad_k():
    with pytest.raises(ValueError):
        oracle.topk(torch.rand(4), 5)


# ---------------------------------------------------------------- pruned attention
def _sel(n, k, seed):
    return torch.randperm(n, generator=torch.Generator().manual_seed(seed))[:k].sort().values.int()


def test_tau_one_reproduces_dense_bit_for_bit():
    q, K, V = _case(31, 100)
    idx = torch.arange(70, dtype=torch.int32)
    for acc64 in (False, True):
        assert torch.equal(oracle.sparse(q, K, V, SCALE, 12, 70, idx, acc64), oracle.dense(q, K, V, SCALE, acc64))


def test_pruned_equals_masked_dense_and_compacted_dense():
    q, K, V = _case(32, 140)
    vs, N, k = 9, 100, 17
    idx = _sel(N, k, 5)
    out = oracle.sparse(q, K, V, SCALE, vs, N, idx, acc64=True)
    keep = torch.ones(140, dtype=torch.bool)
    keep[vs:vs + N] = False
    keep[vs + idx.long()] = True
    assert (out - oracle.masked_dense(q, K, V, SCALE, keep)).abs().max() < 1e-6
    ref, _ = _torch_attention(q, K, V, SCALE, keep)
    assert (out.double() - ref).abs().max() < 1e-6
    assert torch.equal(oracle.sparse(q, K, V, SCALE, vs, N, idx), oracle.dense(q, K[keep], V[keep], SCALE))


def test_pruned_ignores_order_and_unselected_rows():
    q, K, V = _case(33, 60)
    idx = _sel(40, 8, 2)
    a = oracle.sparse(q, K, V, SCALE, 5, 40, idx)
    b = oracle.sparse(q, K, V, SCALE, 5, 40, idx.flip(0))
    assert torch.equal(a, b)
    K2, V2 = K.clone(), V.clone()
    drop = torch.ones(40, dtype=torch.bool)
    drop[idx.long()] = False
    K2[5:45][drop] = float("nan")
    V2[5:45][drop] = float("nan")
    assert torch.equal(a, oracle.sparse(q, K2, V2, SCALE, 5, 40, idx))


def test_k_zero_is_dense_over_text_only():
    q, K, V = _case(34, 70)
    out = oracle.sparse(q, K, V, SCALE, 6, 50, torch.empty(0, dtype=torch.int32))
    keep = torch.ones(70, dtype=torch.bool)
    keep[6:56] = False
    assert torch.equal(out, oracle.dense(q, K[keep], V[keep], SCALE))


def test_empty_kept_set_and_bad_indices_are_errors():
    q, K, V = _case(35, 30)
    with pytest.raises(ValueError):
        oracle.sparse(q, K, V, SCALE, 0, 30, torch.empty(0, dtype=torch.int32))
    with pytest.raises(ValueError):
        oracle.sparse(q, K, V, SCALE, 0, 20, torch.tensor([20], dtype=torch.int32))

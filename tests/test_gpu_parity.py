"""GPU parity: every C-ABI entry point against the CPU oracle, element by element, on seeded
inputs that span several tiles and ragged tails. Tolerances: index lists bit-exact on identical
scores; end-to-end selections may differ only at near-ties (relative gap < 1e-5); outputs within
max-abs 1e-2 / mean-abs 1e-3 of the fp32 oracle (the stated bound) and, since both sides
accumulate in fp32 from the same bf16 bytes, within 1e-4 max-abs in practice (asserted too)."""
import math

import pytest
import torch

import oracle
from harness import SCALE, make_case

pytestmark = pytest.mark.gpu

# FASTOCR_CLUSTER_MAX_ROWS=0 (a tuning knob read when a context is created) turns the merge inside
# thread-block clusters off; the tests that assert which path ran follow the knob.
import os
CLUSTERS_ON = int(os.environ.get("FASTOCR_CLUSTER_MAX_ROWS", "6")) > 0

MAX_ABS, MEAN_ABS = 1e-2, 1e-3      # stated tolerance for bf16 K/V/Q against the fp32 oracle
TIGHT = 1e-4                        # what fp32 accumulation on both sides actually delivers


@pytest.fixture(scope="module")
def fo():
    import paper_2605_17447_b200 as f
    return f


@pytest.fixture(scope="module")
def ctx(fo):
    c = fo.Context(max_batch=8, num_q_heads=64, num_kv_heads=8, max_seq_len=40000, max_vis_len=32768)
    yield c
    assert c.device_faults() == 0
    c.close()


def _check_out(got, ref):
    err = (got.float().cpu() - ref).abs()
    assert err.max() <= MAX_ABS and err.mean() <= MEAN_ABS
    assert err.max() <= TIGHT, float(err.max())


def _oracle_dense(case, acc64=True):
    return torch.stack([oracle.dense(*case.seq(b), SCALE, acc64) for b in range(case.B)])


def _oracle_scores(case, acc64=True):
    return [oracle.scores(case.q[b], case.seq(b)[1], SCALE, case.vis_start[b], case.vis_len[b], acc64) for b in range(case.B)]


SHAPES = [
    dict(spans=[(16, 1024, 48)]),                                   # config 0
    dict(spans=[(3, 50, 2), (0, 333, 0), (7, 1, 100), (40, 0, 0)]),  # ragged, image at the front, no image
    dict(spans=[(16, 2500, 77), (16, 4097, 130)]),                  # several splits + ragged tail
    dict(spans=[(5, 700, 9), (1, 90, 3)], H=64, Hkv=8),             # 72B-shaped group of 8
    dict(spans=[(2, 130, 5)], H=4, Hkv=2),
    dict(spans=[(2, 40, 5)], H=3, Hkv=3),
]


@pytest.mark.parametrize("shape", range(len(SHAPES)))
@pytest.mark.parametrize("paged", [False, True])
def test_dense_and_fused_scores_match_oracle(fo, ctx, shape, paged):
    case = make_case(100 + shape, page_size=16 if paged else 0, **SHAPES[shape])
    kv = case.device_view(poison=True)
    q = case.q.cuda()
    out = torch.empty(case.B, case.H, 128, dtype=torch.float32, device="cuda")
    nmax = max(max(case.vis_len), 1)
    sc = torch.full((case.B, nmax + 3), -7.0, dtype=torch.float32, device="cuda")
    before = fo.cluster_launch_count()
    fo.fastocr_dense_decode_attn(ctx, kv, q, out, scores_out=sc)
    # a single sequence leaves most SMs empty anyway: each (sequence, KV head) unit is then one cluster of
    # 16 CTAs and merges inside it (some units have fewer than 16 rows: CTAs without work in the cluster)
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    assert fo.cluster_launch_count() == before + (1 if CLUSTERS_ON and 2 * 16 * case.B * case.Hkv <= sms else 0)
    _check_out(out, _oracle_dense(case))
    # fp32-accumulating oracle too (the stated reference)
    err32 = (out.cpu() - _oracle_dense(case, acc64=False)).abs()
    assert err32.max() <= MAX_ABS and err32.mean() <= MEAN_ABS
    ref = _oracle_scores(case)
    sc = sc.cpu()
    for b in range(case.B):
        n = case.vis_len[b]
        r = ref[b][0]
        assert ((sc[b, :n] - r).abs() <= 2e-5 * r + 1e-12).all()
        assert (sc[b, n:] == -7.0).all()                            # padding untouched
    # bf16 output path
    outb = torch.empty(case.B, case.H, 128, dtype=torch.bfloat16, device="cuda")
    fo.fastocr_dense_decode_attn(ctx, kv, q, outb)
    assert torch.equal(outb.cpu(), out.cpu().to(torch.bfloat16))


@pytest.mark.parametrize("shape", [0, 1, 2, 3])
def test_focal_scores_standalone_and_image_mass(fo, ctx, shape):
    case = make_case(200 + shape, **SHAPES[shape])
    kv = case.device_view()
    nmax = max(max(case.vis_len), 1)
    sc = torch.zeros(case.B, nmax, dtype=torch.float32, device="cuda")
    mass = torch.zeros(case.B, dtype=torch.float32, device="cuda")
    fo.fastocr_focal_scores(ctx, kv, case.q.cuda(), sc, image_mass_out=mass)
    ref = _oracle_scores(case)
    for b in range(case.B):
        n = case.vis_len[b]
        r = ref[b][0]
        assert ((sc[b, :n].cpu() - r).abs() <= 2e-5 * r + 1e-12).all()
        assert abs(float(mass[b]) - ref[b][1]) <= 1e-5
    # the fused and the stand-alone scores are the same computation
    out = torch.empty(case.B, case.H, 128, dtype=torch.float32, device="cuda")
    sc2 = torch.zeros_like(sc)
    fo.fastocr_dense_decode_attn(ctx, kv, case.q.cuda(), out, scores_out=sc2)
    assert torch.equal(sc, sc2)


def _topk_gpu(fo, ctx, scores, ns, ks, k_stride=None):
    B = len(ns)
    k_stride = k_stride or max(max(ks), 1)
    idx = torch.full((B, k_stride), -1, dtype=torch.int32, device="cuda")
    fo.fastocr_select_topk(ctx, scores.cuda().contiguous(), torch.tensor(ns, dtype=torch.int32, device="cuda"),
                           torch.tensor(ks, dtype=torch.int32, device="cuda"), idx, max(max(ns), 1))
    return idx.cpu()


@pytest.mark.parametrize("n", [1, 31, 1000, 4097, 32768])
def test_topk_bit_exact_on_identical_scores(fo, ctx, n):
    g = torch.Generator().manual_seed(n)
    rows = [torch.rand(n, generator=g) * 1e-3,                                   # softmax-like magnitudes
            torch.randint(0, 5, (n,), generator=g).float() / 8,                  # heavy ties
            torch.full((n,), 0.125),                                            # all equal
            torch.randn(n, generator=g),                                        # negatives
            (torch.rand(n, generator=g) * 1e-30)]                               # tiny / denormal-adjacent
    special = torch.randn(n, generator=g)
    if n >= 8:
        special[[0, 1, 2, 3, 4, 5]] = torch.tensor([0.0, -0.0, float("nan"), float("inf"), float("-inf"), float("nan")])
    rows.append(special)
    for ki, k in enumerate(sorted({0, 1, min(52, n), n // 2, n - 1, n})):
        if k < 0:
            continue
        scores = torch.stack(rows)
        ks = [k] * len(rows)
        got = _topk_gpu(fo, ctx, scores, [n] * len(rows), ks)
        for r in range(len(rows)):
            assert got[r, :k].tolist() == oracle.topk(rows[r], k).tolist(), (n, k, r)
            assert (got[r, k:] == -1).all()


def test_topk_ragged_batch_and_clamped_k(fo, ctx):
    g = torch.Generator().manual_seed(9)
    ns, ks = [100, 5000, 1, 777], [5, 250, 1, 9999]           # last k exceeds N: clamped to N
    scores = torch.rand(4, 5003, generator=g)
    got = _topk_gpu(fo, ctx, scores, ns, ks, k_stride=1000)
    for b in range(4):
        k = min(ks[b], ns[b], 1000)
        assert got[b, :k].tolist() == oracle.topk(scores[b, :ns[b]], k).tolist()


@pytest.mark.parametrize("shape", range(len(SHAPES)))
@pytest.mark.parametrize("paged", [False, True])
def test_sparse_matches_oracle(fo, ctx, shape, paged):
    case = make_case(300 + shape, page_size=16 if paged else 0, **SHAPES[shape])
    kv = case.device_view(poison=True)
    g = torch.Generator().manual_seed(shape)
    ks = [oracle.kept_count(n, 0.05) for n in case.vis_len]
    kmax = max(max(ks), 1)
    idx = torch.zeros(case.B, kmax, dtype=torch.int32)
    for b in range(case.B):
        idx[b, :ks[b]] = torch.randperm(case.vis_len[b], generator=g)[:ks[b]].sort().values.int()
    out = torch.empty(case.B, case.H, 128, dtype=torch.float32, device="cuda")
    fo.fastocr_sparse_decode_attn(ctx, kv, case.q.cuda(), idx.cuda(), torch.tensor(ks, dtype=torch.int32, device="cuda"), out,
                                  max_kept=max(k + s - n for k, s, n in zip(ks, case.seq_len, case.vis_len)))
    ref = torch.stack([oracle.sparse(*case.seq(b), SCALE, case.vis_start[b], case.vis_len[b], idx[b, :ks[b]], True)
                       if ks[b] + case.seq_len[b] - case.vis_len[b] > 0 else torch.zeros(case.H, 128)
                       for b in range(case.B)])
    _check_out(out, ref)


# Short pruned passes over sequences of similar length run one thread-block cluster per unit and
# merge a unit's pieces through distributed shared memory: cluster sizes up to 16, a shorter
# sequence whose units leave CTAs of their cluster without rows, the 8-head group, paged caches.
CLUSTER_CASES = [
    dict(spans=[(16, 4000, 48)], k=[200]),                          # 264 tokens: 9 rows, 9 CTAs per unit
    dict(spans=[(10, 3000, 22), (10, 2500, 22)], k=[224, 192]),     # 8 and 7 rows on clusters of 8: one idle CTA each
    dict(spans=[(30, 6000, 40)], k=[440], H=64, Hkv=8),             # 510 tokens: 16 rows, clusters of 16
    dict(spans=[(5, 900, 5), (6, 880, 5), (5, 910, 4), (4, 905, 6)], k=[90, 88, 91, 90]),   # 4 rows: clusters of 4
]


@pytest.mark.parametrize("case_no", range(len(CLUSTER_CASES)))
@pytest.mark.parametrize("paged", [False, True])
def test_sparse_cluster_merge_matches_oracle(fo, ctx, case_no, paged):
    spec = dict(CLUSTER_CASES[case_no])
    ks = spec.pop("k")
    case = make_case(350 + case_no, page_size=16 if paged else 0, **spec)
    kv = case.device_view(poison=True)
    g = torch.Generator().manual_seed(case_no)
    idx = torch.zeros(case.B, max(ks), dtype=torch.int32)
    for b in range(case.B):
        idx[b, :ks[b]] = torch.randperm(case.vis_len[b], generator=g)[:ks[b]].sort().values.int()
    kd = torch.tensor(ks, dtype=torch.int32, device="cuda")
    max_kept = max(k + s - n for k, s, n in zip(ks, case.seq_len, case.vis_len))
    ref = torch.stack([oracle.sparse(*case.seq(b), SCALE, case.vis_start[b], case.vis_len[b], idx[b, :ks[b]], True)
                       for b in range(case.B)])
    q = case.q.cuda()
    out = torch.full((case.B, case.H, 128), 7.0, dtype=torch.float32, device="cuda")
    before = fo.cluster_launch_count()
    fo.fastocr_sparse_decode_attn(ctx, kv, q, idx.cuda(), kd, out, max_kept=max_kept)
    assert fo.cluster_launch_count() == before + (1 if CLUSTERS_ON else 0)       # the path under test is the one that ran
    _check_out(out, ref)
    # the same inside a decode step, three pruned layers on last step's set: as one group launch (the
    # library's default), and, with group launches switched off, as three cluster launches from a launch plan
    for group_layers in ("32", "1"):
        saved = os.environ.get("FASTOCR_GROUP_LAYERS")
        os.environ["FASTOCR_GROUP_LAYERS"] = group_layers        # read when a context is created
        c2 = fo.Context(max_batch=8, num_q_heads=64, num_kv_heads=8, max_seq_len=40000, max_vis_len=32768)
        if saved is None:
            del os.environ["FASTOCR_GROUP_LAYERS"]
        else:
            os.environ["FASTOCR_GROUP_LAYERS"] = saved
        out3 = torch.full((3, case.B, case.H, 128), 7.0, dtype=torch.float32, device="cuda")
        before = fo.cluster_launch_count()
        assert fo.fastocr_decode_step(c2, [kv, kv, kv], torch.stack([q, q, q]), out3, [False, False, False], kd,
                                      idx.cuda().clone(), True, max(case.vis_len), max_kept=max_kept)
        if group_layers == "1":
            assert fo.cluster_launch_count() == before + (3 if CLUSTERS_ON else 0)
        for l in range(3):
            _check_out(out3[l], ref)
        assert c2.device_faults() == 0
        c2.close()


@pytest.mark.parametrize("seed", range(12))
def test_sparse_random_batches_match_oracle(fo, ctx, seed):
    """Seeded random batches (1-8 sequences, similar or very different lengths, any kept fraction, paged
    or not, with and without the caller's bound on kept tokens): whichever way the kernel hands out
    the rows (equal parts, one CTA per unit, equal ranges; merged in clusters or through global
    memory), the result is the oracle's."""
    g = torch.Generator().manual_seed(1000 + seed)
    ri = lambda lo, hi: int(torch.randint(lo, hi + 1, (1,), generator=g))
    B = ri(1, 8)
    similar = seed % 2 == 0
    n0 = ri(64, 3000)
    spans = []
    for _ in range(B):
        n = max(1, n0 + ri(-n0 // 20, n0 // 20)) if similar else ri(1, 3000)
        spans.append((ri(0, 40), n, ri(0, 120)))
    tau = [0.02, 0.05, 0.1, 0.3, 0.6, 1.0][seed % 6]
    heads = dict(H=64, Hkv=8) if seed % 4 == 3 else {}
    case = make_case(1100 + seed, spans=spans, page_size=16 if seed % 3 == 0 else 0, **heads)
    kv = case.device_view(poison=True)
    ks = [oracle.kept_count(n, tau) for n in case.vis_len]
    idx = torch.zeros(case.B, max(max(ks), 1), dtype=torch.int32)
    for b in range(case.B):
        idx[b, :ks[b]] = torch.randperm(case.vis_len[b], generator=g)[:ks[b]].sort().values.int()
    attended = [k + s - n for k, s, n in zip(ks, case.seq_len, case.vis_len)]
    ref = torch.stack([oracle.sparse(*case.seq(b), SCALE, case.vis_start[b], case.vis_len[b], idx[b, :ks[b]], True)
                       if attended[b] > 0 else torch.zeros(case.H, 128) for b in range(case.B)])
    kd = torch.tensor(ks, dtype=torch.int32, device="cuda")
    for max_kept in (max(attended), 0):
        out = torch.full((case.B, case.H, 128), 7.0, dtype=torch.float32, device="cuda")
        fo.fastocr_sparse_decode_attn(ctx, kv, case.q.cuda(), idx.cuda(), kd, out, max_kept=max_kept)
        _check_out(out, ref)


def test_sparse_tau_one_equals_dense_and_tau_zero_is_text_only(fo, ctx):
    case = make_case(401, spans=[(16, 600, 40), (4, 333, 9)])
    kv = case.device_view()
    q = case.q.cuda()
    dense = torch.empty(case.B, case.H, 128, dtype=torch.float32, device="cuda")
    fo.fastocr_dense_decode_attn(ctx, kv, q, dense)
    idx = torch.zeros(case.B, 600, dtype=torch.int32)
    for b in range(case.B):
        idx[b, :case.vis_len[b]] = torch.arange(case.vis_len[b])
    out = torch.empty_like(dense)
    fo.fastocr_sparse_decode_attn(ctx, kv, q, idx.cuda(), torch.tensor(case.vis_len, dtype=torch.int32, device="cuda"), out)
    assert (out - dense).abs().max() <= 1e-5                       # same rows, possibly another split
    fo.fastocr_sparse_decode_attn(ctx, kv, q, idx.cuda(), torch.zeros(case.B, dtype=torch.int32, device="cuda"), out)
    ref = torch.stack([oracle.sparse(*case.seq(b), SCALE, case.vis_start[b], case.vis_len[b],
                                     torch.empty(0, dtype=torch.int32), True) for b in range(case.B)])
    _check_out(out, ref)


def test_sequence_with_nothing_to_attend_gets_zeros(fo, ctx):
    """A sequence without text tokens and with a kept count of 0 attends nothing: its outputs are
    zeros, the others are unaffected; stand-alone and inside a decode step (whose launch plan must
    step aside for such a batch)."""
    case = make_case(450, spans=[(4, 200, 10), (0, 150, 0), (3, 90, 5)])
    kv = case.device_view(poison=True)
    q = case.q.cuda()
    ks = [oracle.kept_count(case.vis_len[0], 0.1), 0, oracle.kept_count(case.vis_len[2], 0.1)]
    g = torch.Generator().manual_seed(5)
    idx = torch.zeros(case.B, max(ks), dtype=torch.int32)
    for b in range(case.B):
        idx[b, :ks[b]] = torch.randperm(case.vis_len[b], generator=g)[:ks[b]].sort().values.int()
    kd = torch.tensor(ks, dtype=torch.int32, device="cuda")
    ref = torch.stack([oracle.sparse(*case.seq(b), SCALE, case.vis_start[b], case.vis_len[b], idx[b, :ks[b]], True)
                       if b != 1 else torch.zeros(case.H, 128) for b in range(case.B)])
    out = torch.full((case.B, case.H, 128), 7.0, dtype=torch.float32, device="cuda")
    fo.fastocr_sparse_decode_attn(ctx, kv, q, idx.cuda(), kd, out)
    _check_out(out, ref)
    assert float(out[1].abs().max()) == 0.0
    out3 = torch.full((3, case.B, case.H, 128), 7.0, dtype=torch.float32, device="cuda")
    fix = idx.cuda().clone()
    assert fo.fastocr_decode_step(ctx, [kv, kv, kv], torch.stack([q, q, q]), out3, [False, False, False], kd, fix, True,
                                  max(case.vis_len))
    for l in range(3):
        _check_out(out3[l], ref)
        assert float(out3[l, 1].abs().max()) == 0.0


def _near_tie_only(gpu_idx, ref_idx, ref_scores, k):
    """Selections may differ only in tokens whose oracle score is within 1e-5 (relative) of the
    oracle's k-th score."""
    a, b = set(gpu_idx.tolist()), set(ref_idx.tolist())
    if a == b:
        return True
    kth = float(torch.sort(ref_scores, descending=True).values[k - 1])
    return all(abs(float(ref_scores[i]) - kth) <= 1e-5 * abs(kth) for i in a ^ b)


@pytest.mark.parametrize("shape", [0, 1, 2, 3])
def test_end_to_end_selection_then_sparse(fo, ctx, shape):
    """dense+scores -> top-k -> pruned attention on the same layer, all on the GPU, against the
    oracle's own chain (config 0's 'scored and attended' layer among the shapes)."""
    case = make_case(500 + shape, **SHAPES[shape])
    kv = case.device_view()
    q = case.q.cuda()
    nmax = max(max(case.vis_len), 1)
    ks = [oracle.kept_count(n, 0.05) for n in case.vis_len]
    kmax = max(max(ks), 1)
    sc = torch.zeros(case.B, nmax, dtype=torch.float32, device="cuda")
    dense = torch.empty(case.B, case.H, 128, dtype=torch.float32, device="cuda")
    idx = torch.zeros(case.B, kmax, dtype=torch.int32, device="cuda")
    kd = torch.tensor(ks, dtype=torch.int32, device="cuda")
    out = torch.empty_like(dense)
    fo.fastocr_dense_decode_attn(ctx, kv, q, dense, scores_out=sc)
    fo.fastocr_select_topk(ctx, sc, kv.vis_len, kd, idx, nmax)
    fo.fastocr_sparse_decode_attn(ctx, kv, q, idx, kd, out)
    idx_c = idx.cpu()
    for b in range(case.B):
        if ks[b] == 0:
            continue
        ref_sc, _ = oracle.scores(case.q[b], case.seq(b)[1], SCALE, case.vis_start[b], case.vis_len[b], True)
        ref_idx = oracle.topk(ref_sc, ks[b])
        assert _near_tie_only(idx_c[b, :ks[b]], ref_idx, ref_sc, ks[b])
        assert idx_c[b, :ks[b]].tolist() == sorted(set(idx_c[b, :ks[b]].tolist()))       # ascending, distinct
        # bit-exact against the oracle's selection rule applied to the GPU's own scores
        assert idx_c[b, :ks[b]].tolist() == oracle.topk(sc[b, :case.vis_len[b]].cpu(), ks[b]).tolist()
        ref_out = oracle.sparse(*case.seq(b), SCALE, case.vis_start[b], case.vis_len[b], idx_c[b, :ks[b]], True)
        _check_out(out[b], ref_out)


def test_fixation_window_is_selected_on_config0(fo, ctx):
    """Sanity of the workload recipe: the 3x3 window the query was built from is inside the top 5%."""
    from workloads import get_config
    cfg = get_config("cfg0")
    case = make_case(cfg.seed, [(cfg.text_before[0], cfg.vis_len[0], cfg.text_after[0])], grid_w=32)
    sc, _ = oracle.scores(case.q[0], case.seq(0)[1], SCALE, 16, 1024, True)
    k = oracle.kept_count(1024, cfg.tau)
    assert k == 52
    sel = set(oracle.topk(sc, k).tolist())
    top9 = set(torch.topk(sc, 9).indices.tolist())
    assert len(top9 & sel) == 9


@pytest.mark.parametrize("paged,spans", [(False, [(6, 300, 20), (3, 170, 41)]), (True, [(6, 300, 20), (3, 170, 41)]),
                                         (False, [(5, 200, 30)] * 3), (True, [(5, 200, 30)] * 3)])
def test_decode_step_matches_algorithm_trace(fo, ctx, paged, spans):
    """Ragged and uniform batches (the latter get valid launch-plan records), contiguous and paged caches."""
    L = 5
    base = make_case(600, spans, page_size=16 if paged else 0)
    from workloads import make_kv, normal_bf16, stream_key
    layers_cpu, views = [], []
    shared = None                                        # one set of length arrays for all layers, as a caller
    for l in range(L):                                   # would have (that is what makes a launch plan usable)
        K, V = make_kv(600, l, base.B, max(base.seq_len), base.Hkv, 128)
        q = normal_bf16(stream_key(600, 55, l), (base.B, base.H, 128))
        c = type(base)(base.B, base.H, base.Hkv, base.seq_len, base.vis_start, base.vis_len, K, V, q,
                       base.page_size, base.block_table, base.num_pages)
        layers_cpu.append(c)
        v = c.device_view()
        if shared is None:
            shared = (v.seq_len, v.vis_start, v.vis_len)
        v = fo.KVView(v.k, v.v, shared[0], shared[1], shared[2], base.H, max(base.seq_len), SCALE,
                      block_table=v.block_table if paged else None)
        views.append(v)
    q_all = torch.stack([c.q for c in layers_cpu]).cuda()
    ks = [oracle.kept_count(n, 0.1) for n in base.vis_len]
    kd = torch.tensor(ks, dtype=torch.int32, device="cuda")
    fix = torch.full((base.B, max(ks)), -1, dtype=torch.int32, device="cuda")
    for focal, steps in (([2], 2), ([0, 3], 1), ([], 2)):
        is_focal = [l in focal for l in range(L)]
        have = False
        f_last = [None] * base.B
        fix.fill_(-1)
        for _ in range(steps):
            out = torch.empty(L, base.B, base.H, 128, dtype=torch.float32, device="cuda")
            have = fo.fastocr_decode_step(ctx, views, q_all, out, is_focal, kd, fix, have, max(base.vis_len))
            assert have
            for b in range(base.B):
                tr = oracle.decode_step([c.seq(b) for c in layers_cpu], focal, f_last[b], base.vis_start[b],
                                        base.vis_len[b], 0.1, SCALE, acc64=True)
                for l in range(L):
                    _check_out(out[l, b], tr.outputs[l])
                assert fix[b, :ks[b]].cpu().tolist() == tr.f_last.tolist()
                f_last[b] = tr.f_last


@pytest.mark.parametrize("batch,n", [(2, 16384), (5, 4100), (1, 2048), (1, 32768), (3, 32768), (20, 16384)])
def test_decode_step_selection_equals_separate_calls(fo, batch, n):
    """The decode step's selection kernel forms the scores itself, with a cluster of up to 8 CTAs per
    sequence for small batches; it must select exactly what scoring + selection as separate calls do.
    (The last three shapes take the variant that splits the selection itself over the cluster:
    32768 keys on clusters of 8, 16384 keys on clusters of 4.)"""
    from workloads import make_kv, normal_bf16, stream_key
    dev = "cuda"
    H, Hkv, T = 28, 4, 40
    S = n + T
    K, V = make_kv(900 + batch, 0, batch, S, Hkv, 128, dev)
    q = (normal_bf16(stream_key(901, batch), (batch, H, 128), dev).float() * 3).to(torch.bfloat16)
    i32 = lambda x: torch.tensor(x, dtype=torch.int32, device=dev)
    vis = [n - 7 * b for b in range(batch)]                      # ragged image spans
    kv = fo.KVView(K, V, i32([S - 7 * b for b in range(batch)]), i32([8] * batch), i32(vis), H, S, SCALE)
    ks = [oracle.kept_count(v, 0.05) for v in vis]
    kd = i32(ks)
    c2 = fo.Context(batch, H, Hkv, S, n)
    dense = torch.empty(batch, H, 128, dtype=torch.float32, device=dev)
    sc = torch.zeros(batch, n, dtype=torch.float32, device=dev)
    idx = torch.full((batch, max(ks)), -1, dtype=torch.int32, device=dev)
    fo.fastocr_dense_decode_attn(c2, kv, q, dense, scores_out=sc)
    fo.fastocr_select_topk(c2, sc, kv.vis_len, kd, idx, n)
    fix = torch.full_like(idx, -1)
    out = torch.empty(1, batch, H, 128, dtype=torch.float32, device=dev)
    assert fo.fastocr_decode_step(c2, [kv], q[None], out, [True], kd, fix, False, n)
    torch.cuda.synchronize()
    assert torch.equal(fix, idx) and torch.equal(out[0], dense)
    for b in range(batch):                                        # and both are the oracle's choice on these scores
        assert idx[b, :ks[b]].cpu().tolist() == oracle.topk(sc[b, :vis[b]].cpu(), ks[b]).tolist()
    c2.close()


def test_argument_errors_are_reported_not_launched(fo, ctx):
    case = make_case(700, [(4, 64, 4)])
    kv = case.device_view()
    q = case.q.cuda()
    out = torch.empty(1, 28, 128, dtype=torch.float32, device="cuda")
    before = fo.launch_count()
    small = fo.Context(max_batch=1, num_q_heads=28, num_kv_heads=4, max_seq_len=32, max_vis_len=64)
    with pytest.raises(fo.FastOCRError) as e:                   # 72 cached tokens > the context's 32
        fo.fastocr_dense_decode_attn(small, kv, q, out)
    assert e.value.code == 3
    small.close()
    bad = case.device_view()
    bad.num_q_heads = 36                                        # group of 9: unsupported
    with pytest.raises(fo.FastOCRError) as e:
        fo.fastocr_dense_decode_attn(ctx, bad, q, out)
    assert e.value.code == 2
    bad = case.device_view()
    bad.sm_scale = 0.0
    with pytest.raises(fo.FastOCRError) as e:
        fo.fastocr_dense_decode_attn(ctx, bad, q, out)
    assert e.value.code == 1
    with pytest.raises(fo.FastOCRError):
        fo.fastocr_select_topk(ctx, torch.zeros(1, 8, device="cuda"), kv.vis_len, kv.vis_len,
                               torch.zeros(1, 4, dtype=torch.int32, device="cuda"), 99)   # max_vis_len > n_stride
    assert fo.launch_count() == before

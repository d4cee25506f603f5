"""GPU parity of the step-level entry points beyond Algorithm 1's plain post-warm-up step: the warm-up
step (profiling block), per-sequence focal layer sets, the union-of-selections variant, the 64-head
shape inside a decode step, and what the kernels do with device-side lengths, index-list entries and
page ids that lie outside what the host checked. Everything goes through the C ABI and is compared
with the CPU oracle element by element."""
import math

import pytest
import torch

import oracle
from harness import SCALE, make_case, make_layer_stack

pytestmark = pytest.mark.gpu

MAX_ABS, MEAN_ABS, TIGHT = 1e-2, 1e-3, 1e-4


@pytest.fixture(scope="module")
def fo():
    import paper_2605_17447_b200 as f
    return f


@pytest.fixture(scope="module")
def ctx(fo):
    c = fo.Context(max_batch=8, num_q_heads=64, num_kv_heads=8, max_seq_len=8192, max_vis_len=6000)
    yield c
    c.close()


def _check_out(got, ref):
    err = (got.float().cpu() - ref).abs()
    assert err.max() <= MAX_ABS and err.mean() <= MEAN_ABS
    assert err.max() <= TIGHT, float(err.max())


def test_warmup_step_records_eq1_and_keeps_dense_outputs(fo, ctx):
    """Algorithm 1's profiling block: w steps, every layer dense, r per layer and sequence from the same
    pass; the focal layer sets that follow (per sequence) equal the oracle's."""
    L, w = 4, 3
    spans = [(6, 300, 20), (3, 170, 41), (9, 512, 7)]
    ratios_gpu = torch.zeros(w, L, len(spans), dtype=torch.float32)
    ratios_ref = torch.zeros(w, L, len(spans), dtype=torch.float64)
    for t in range(w):
        cases, views, q_all = make_layer_stack(1300 + t, spans, L)
        out = torch.empty(L, len(spans), 28, 128, dtype=torch.float32, device="cuda")
        r = torch.full((L, len(spans)), -1.0, dtype=torch.float32, device="cuda")
        fo.fastocr_warmup_step(ctx, views, q_all.cuda(), out, r)
        ratios_gpu[t] = r.cpu()
        for b in range(len(spans)):
            outs, rr = oracle.warmup_step([c.seq(b) for c in cases], cases[0].vis_start[b], cases[0].vis_len[b], SCALE, acc64=True)
            for l in range(L):
                _check_out(out[l, b], outs[l])
                ratios_ref[t, l, b] = rr[l]
    assert float((ratios_gpu.double() - ratios_ref).abs().max()) <= 1e-5
    for b in range(len(spans)):
        mean_gpu = ratios_gpu[:, :, b].double().mean(dim=0).tolist()
        assert fo.focal_layers(mean_gpu, 0.5, 1) == oracle.profile_focal_layers(ratios_ref[:, :, b].tolist(), 0.5, 1)
    # the single-layer call gives the same ratio with or without the score array
    cases, views, q_all = make_layer_stack(1300, spans, 1)
    out = torch.empty(len(spans), 28, 128, dtype=torch.float32, device="cuda")
    sc = torch.zeros(len(spans), 512, dtype=torch.float32, device="cuda")
    m1 = torch.zeros(len(spans), dtype=torch.float32, device="cuda")
    m2 = torch.zeros_like(m1)
    fo.fastocr_dense_decode_attn(ctx, views[0], q_all[0].cuda(), out, image_mass_out=m1)
    fo.fastocr_dense_decode_attn(ctx, views[0], q_all[0].cuda(), out, scores_out=sc, image_mass_out=m2)
    assert torch.equal(m1, m2) and torch.equal(m1.cpu(), ratios_gpu[0, 0])
    assert ctx.device_faults() == 0


@pytest.mark.parametrize("paged", [False, True])
def test_decode_step_with_per_sequence_focal_sets(fo, ctx, paged):
    """Each sequence has its own focal layer set (the paper profiles C per sample): a layer that is focal
    for part of the batch runs as two masked launches. Two consecutive steps, every sequence against
    the oracle run with that sequence's own set."""
    L = 6
    spans = [(6, 300, 20), (3, 170, 41), (5, 222, 9), (2, 260, 30)]
    focal_of = [[2], [1, 3], [], [0, 3]]                      # layer 3 mixed 2:2, layer 0 focal for one sequence only
    matrix = [[l in focal_of[b] for b in range(len(spans))] for l in range(L)]
    cases, views, q_all = make_layer_stack(1400, spans, L, page_size=16 if paged else 0)
    base = cases[0]
    ks = [oracle.kept_count(n, 0.1) for n in base.vis_len]
    kd = torch.tensor(ks, dtype=torch.int32, device="cuda")
    fix = torch.full((base.B, max(ks)), -1, dtype=torch.int32, device="cuda")
    have, f_last = False, [None] * base.B
    for step in range(2):
        out = torch.full((L, base.B, base.H, 128), 7.0, dtype=torch.float32, device="cuda")
        have = fo.fastocr_decode_step(ctx, views, q_all.cuda(), out, matrix, kd, fix, have, max(base.vis_len))
        assert have
        for b in range(base.B):
            tr = oracle.decode_step([c.seq(b) for c in cases], focal_of[b], f_last[b], base.vis_start[b], base.vis_len[b],
                                    0.1, SCALE, acc64=True)
            for l in range(L):
                _check_out(out[l, b], tr.outputs[l])
            assert fix[b, :ks[b]].cpu().tolist() == tr.f_last.tolist()
            f_last[b] = tr.f_last
    assert ctx.device_faults() == 0


@pytest.mark.parametrize("per_seq", [False, True])
def test_decode_step_union_of_selections(fo, ctx, per_seq):
    """The union variant: after a focal layer the kept image set is the union of this step's selections;
    the set carried to the next step stays the deepest focal layer's own."""
    L = 6
    spans = [(6, 300, 20), (3, 170, 41), (4, 280, 11)]
    focal_of = [[1, 3, 4], [2, 4], [1]] if per_seq else [[1, 3, 4]] * 3
    is_focal = [[l in focal_of[b] for b in range(3)] for l in range(L)] if per_seq else [l in focal_of[0] for l in range(L)]
    cases, views, q_all = make_layer_stack(1500, spans, L, q_boost=2.0)
    base = cases[0]
    ks = [oracle.kept_count(n, 0.1) for n in base.vis_len]
    kd = torch.tensor(ks, dtype=torch.int32, device="cuda")
    fix = torch.full((base.B, max(ks)), -1, dtype=torch.int32, device="cuda")
    have, f_last = False, [None] * base.B
    grew = False
    for step in range(2):
        out = torch.full((L, base.B, base.H, 128), 7.0, dtype=torch.float32, device="cuda")
        have = fo.fastocr_decode_step(ctx, views, q_all.cuda(), out, is_focal, kd, fix, have, max(base.vis_len),
                                      max_kept=max(3 * k + s - n for k, s, n in zip(ks, base.seq_len, base.vis_len)), union_sets=True)
        for b in range(base.B):
            tr = oracle.decode_step([c.seq(b) for c in cases], focal_of[b], f_last[b], base.vis_start[b], base.vis_len[b],
                                    0.1, SCALE, acc64=True, union_sets=True)
            for l in range(L):
                _check_out(out[l, b], tr.outputs[l])
            assert fix[b, :ks[b]].cpu().tolist() == tr.f_last.tolist()
            f_last[b] = tr.f_last
            grew = grew or any(u is not None and len(u) > ks[b] for u in tr.used_set)
    assert grew                                                 # the union really was larger than one selection somewhere
    assert ctx.device_faults() == 0


@pytest.mark.parametrize("spans", [[(5, 700, 9), (1, 640, 3)], [(16, 5000, 40), (16, 4800, 56)]])
def test_decode_step_with_64_query_heads(fo, ctx, spans):
    """The 72B-shaped head geometry (64 query / 8 KV heads) through the whole step: the selection kernel
    forms the scores from 64 heads' logits (one token per thread for the short spans, four tokens per
    thread and clusters of CTAs for the long ones)."""
    L = 4
    cases, views, q_all = make_layer_stack(1600, spans, L, H=64, Hkv=8, q_boost=1.5)
    base = cases[0]
    ks = [oracle.kept_count(n, 0.05) for n in base.vis_len]
    kd = torch.tensor(ks, dtype=torch.int32, device="cuda")
    fix = torch.full((base.B, max(ks)), -1, dtype=torch.int32, device="cuda")
    have, f_last = False, [None] * base.B
    for step in range(2):
        out = torch.empty(L, base.B, 64, 128, dtype=torch.float32, device="cuda")
        have = fo.fastocr_decode_step(ctx, views, q_all.cuda(), out, [False, True, False, False], kd, fix, have, max(base.vis_len))
        for b in range(base.B):
            tr = oracle.decode_step([c.seq(b) for c in cases], [1], f_last[b], base.vis_start[b], base.vis_len[b], 0.05, SCALE, acc64=True)
            for l in range(L):
                _check_out(out[l, b], tr.outputs[l])
            assert fix[b, :ks[b]].cpu().tolist() == tr.f_last.tolist()
            f_last[b] = tr.f_last
    assert ctx.device_faults() == 0


def test_kept_count_beyond_the_index_rows_uses_the_row(fo, ctx):
    """k[b] larger than the index list's row length: the first k_stride entries are the set (nothing past
    the row is read), which is not a fault."""
    case = make_case(1700, [(4, 200, 10), (3, 90, 5)])
    kv = case.device_view()
    g = torch.Generator().manual_seed(3)
    k_stride = 12
    idx = torch.stack([torch.randperm(n, generator=g)[:k_stride].sort().values.int() for n in case.vis_len])
    # the buffer really ends after the rows: a read past them would meet the guard values placed behind
    flat = torch.full((2 * k_stride + 64,), 10 ** 6, dtype=torch.int32)
    flat[:2 * k_stride] = idx.flatten()
    dev = flat.cuda()
    out = torch.empty(2, 28, 128, dtype=torch.float32, device="cuda")
    fo.fastocr_sparse_decode_attn(ctx, kv, case.q.cuda(), dev[:2 * k_stride].view(2, k_stride),
                                  torch.tensor([40, 9999], dtype=torch.int32, device="cuda"), out)
    ref = torch.stack([oracle.sparse(*case.seq(b), SCALE, case.vis_start[b], case.vis_len[b], idx[b], True) for b in range(2)])
    _check_out(out, ref)
    assert ctx.device_faults() == 0


def test_device_side_lengths_are_forced_into_range_and_counted(fo, ctx):
    """seq_len / vis_start / vis_len live in device memory, where the host cannot check them. Values outside
    what the host did check are forced into range and counted; the other sequences are unaffected. The
    caches are over-allocated, so that even the unclamped reads would have stayed inside the buffers."""
    case = make_case(1800, [(4, 200, 10), (3, 90, 5), (6, 150, 8)])
    kv = case.device_view(extra_stride=4096)                    # rows far beyond max_seq_len exist (zeros)
    q = case.q.cuda()
    good = torch.stack([oracle.dense(*case.seq(b), SCALE, True) for b in range(3)])
    out = torch.empty(3, 28, 128, dtype=torch.float32, device="cuda")
    i32 = lambda x: torch.tensor(x, dtype=torch.int32, device="cuda")
    assert ctx.device_faults() == 0
    for bad_seq_len, bad_start, bad_len, want in (
            ([214, 98 + 3000, 164], None, None, 1),             # longer than max_seq_len
            ([214, -5, 164], None, None, 3),                    # negative: the span no longer fits either
            (None, [4, -7, 6], None, 1),                        # span starts before the sequence
            (None, None, [200, 5000, 150], 1),                  # span longer than the sequence
            ([10 ** 9, 98, -3], [4, 3, 99999], None, 4)):       # several at once
        view = case.device_view(extra_stride=4096)
        view.max_seq_len = kv.max_seq_len
        if bad_seq_len:
            view.seq_len = i32(bad_seq_len)
        if bad_start:
            view.vis_start = i32(bad_start)
        if bad_len:
            view.vis_len = i32(bad_len)
        out.fill_(7.0)
        fo.fastocr_dense_decode_attn(ctx, view, q, out)
        torch.cuda.synchronize()
        assert ctx.device_faults() == want
        ok = [b for b in range(3) if (not bad_seq_len or bad_seq_len[b] == case.seq_len[b])
              and (not bad_start or bad_start[b] == case.vis_start[b]) and (not bad_len or bad_len[b] == case.vis_len[b])]
        for b in ok:
            _check_out(out[b], good[b])
        assert bool(torch.isfinite(out).all())
    # pruned pass and selection with the same kind of input
    ks = [10, 5, 8]
    g = torch.Generator().manual_seed(1)
    idx = torch.zeros(3, 10, dtype=torch.int32)
    for b in range(3):
        idx[b, :ks[b]] = torch.randperm(case.vis_len[b], generator=g)[:ks[b]].sort().values.int()
    view = case.device_view(extra_stride=4096)
    view.max_seq_len = kv.max_seq_len
    view.seq_len = i32([214, 98 + 3000, 164])
    fo.fastocr_sparse_decode_attn(ctx, view, q, idx.cuda(), i32(ks), out)
    torch.cuda.synchronize()
    assert ctx.device_faults() == 1
    for b in (0, 2):
        _check_out(out[b], oracle.sparse(*case.seq(b), SCALE, case.vis_start[b], case.vis_len[b], idx[b, :ks[b]], True))
    sel = torch.full((3, 10), -1, dtype=torch.int32, device="cuda")
    sc = torch.rand(3, 256, generator=g)
    fo.fastocr_select_topk(ctx, sc.cuda(), i32([200, -4, 150]), i32(ks), sel, 256)   # a negative length selects nothing
    torch.cuda.synchronize()
    assert sel[1].tolist() == [-1] * 10
    for b in (0, 2):
        assert sel[b, :ks[b]].cpu().tolist() == oracle.topk(sc[b, :case.vis_len[b]], ks[b]).tolist()


def test_page_ids_outside_the_pool_are_clamped_and_counted(fo, ctx):
    """A block-table entry beyond num_pages is forced into the pool and counted. The pools hold more pages
    than the view declares, so the unclamped read would have stayed inside the allocation too."""
    case = make_case(1900, [(4, 200, 10), (3, 90, 5)], page_size=16)
    kv = case.device_view()
    q = case.q.cuda()
    declared = kv.k.shape[0]
    spare = torch.zeros(64, 16, 4, 128, dtype=torch.bfloat16, device="cuda")
    bad = fo.KVView(torch.cat([kv.k, spare]), torch.cat([kv.v, spare]), kv.seq_len, kv.vis_start, kv.vis_len, 28,
                    kv.max_seq_len, SCALE, block_table=kv.block_table.clone(), num_pages=declared)
    bad.block_table[1, 2] = declared + 40                        # inside the allocation, outside the declared pool
    bad.block_table[1, 3] = -9
    out = torch.empty(2, 28, 128, dtype=torch.float32, device="cuda")
    assert ctx.device_faults() == 0
    fo.fastocr_dense_decode_attn(ctx, bad, q, out)
    torch.cuda.synchronize()
    assert ctx.device_faults() == 2 * 16 * 4                     # two pages x 16 tokens, looked up once by each of the 4 KV heads' units
    _check_out(out[0], oracle.dense(*case.seq(0), SCALE, True))
    assert bool(torch.isfinite(out).all())


@pytest.mark.parametrize("paged", [False, True])
def test_layers_after_a_selection_with_empty_text_or_empty_selection(fo, ctx, paged):
    """Pruned layers after a focal layer, run as one launch: sequences without text tokens, sequences that
    keep no image token, and a sequence with neither (zeros) must come out right; every other sequence is
    the oracle's pruned attention over the set the focal layer selected."""
    L = 4
    spans = [(4, 200, 10), (0, 150, 0), (3, 90, 5), (0, 64, 0), (7, 130, 0)]
    ks = [20, 15, 0, 0, 13]                                      # sequence 1: no text; 2: nothing kept; 3: neither
    cases, views, q_all = make_layer_stack(2000, spans, L, page_size=16 if paged else 0, q_boost=1.5)
    base = cases[0]
    kd = torch.tensor(ks, dtype=torch.int32, device="cuda")
    fix = torch.full((base.B, max(ks)), -1, dtype=torch.int32, device="cuda")
    out = torch.full((L, base.B, base.H, 128), 7.0, dtype=torch.float32, device="cuda")
    assert fo.fastocr_decode_step(ctx, views, q_all.cuda(), out, [True, False, False, False], kd, fix, False, max(base.vis_len))
    torch.cuda.synchronize()
    for b in range(base.B):
        q0, K0, V0 = cases[0].seq(b)
        _check_out(out[0, b], oracle.dense(q0, K0, V0, SCALE, True))
        sel = fix[b, :ks[b]].cpu()
        if ks[b]:
            sc, _ = oracle.scores(q0, K0, SCALE, base.vis_start[b], base.vis_len[b], True)
            ref_sel = oracle.topk(sc, ks[b])
            kth = float(torch.sort(sc, descending=True).values[ks[b] - 1])
            assert all(abs(float(sc[i]) - kth) <= 1e-5 * kth for i in set(sel.tolist()) ^ set(ref_sel.tolist()))
        for l in range(1, L):
            if ks[b] + base.seq_len[b] - base.vis_len[b] == 0:
                assert float(out[l, b].abs().max()) == 0.0
            else:
                _check_out(out[l, b], oracle.sparse(*cases[l].seq(b), SCALE, base.vis_start[b], base.vis_len[b], sel, True))
    assert ctx.device_faults() == 0


def test_a_run_of_pruned_layers_longer_than_one_launch_takes(fo, ctx):
    """35 consecutive pruned layers on a carried set: the run is cut into a launch of 32 layers and one of 3
    (the second starts while the first drains); every layer against the oracle."""
    L = 35
    spans = [(6, 300, 20), (3, 170, 41)]
    cases, views, q_all = make_layer_stack(2200, spans, L)
    base = cases[0]
    ks = [oracle.kept_count(n, 0.1) for n in base.vis_len]
    g = torch.Generator().manual_seed(4)
    fix = torch.zeros(base.B, max(ks), dtype=torch.int32)
    for b in range(base.B):
        fix[b, :ks[b]] = torch.randperm(base.vis_len[b], generator=g)[:ks[b]].sort().values.int()
    out = torch.full((L, base.B, base.H, 128), 7.0, dtype=torch.float32, device="cuda")
    before = fo.launch_count()
    assert fo.fastocr_decode_step(ctx, views, q_all.cuda(), out, [False] * L, torch.tensor(ks, dtype=torch.int32, device="cuda"),
                                  fix.cuda(), True, max(base.vis_len))
    assert fo.launch_count() - before == 2
    for l in range(L):
        for b in range(base.B):
            _check_out(out[l, b], oracle.sparse(*cases[l].seq(b), SCALE, base.vis_start[b], base.vis_len[b], fix[b, :ks[b]], True))
    assert ctx.device_faults() == 0


@pytest.mark.parametrize("H,Hkv", [(3, 3), (4, 2), (16, 4), (8, 1), (6, 2), (10, 2), (12, 2)])
def test_decode_step_other_group_sizes(fo, ctx, H, Hkv):
    """GQA groups of 1, 2, 4, 8, 3, 5 and 6 (12 / 2: the 1.7B OCR model's shape) query heads per KV head through the whole step (runs of pruned layers as
    one launch, a focal layer in between), paged cache, ragged batch."""
    L = 5
    spans = [(6, 300, 20), (0, 170, 41), (5, 64, 0)]
    cases, views, q_all = make_layer_stack(2300 + H, spans, L, H=H, Hkv=Hkv, page_size=16, q_boost=1.5)
    base = cases[0]
    ks = [oracle.kept_count(n, 0.1) for n in base.vis_len]
    kd = torch.tensor(ks, dtype=torch.int32, device="cuda")
    fix = torch.full((base.B, max(ks)), -1, dtype=torch.int32, device="cuda")
    have, f_last = False, [None] * base.B
    for step in range(2):
        out = torch.full((L, base.B, H, 128), 7.0, dtype=torch.float32, device="cuda")
        have = fo.fastocr_decode_step(ctx, views, q_all.cuda(), out, [False, False, True, False, False], kd, fix, have, max(base.vis_len))
        for b in range(base.B):
            tr = oracle.decode_step([c.seq(b) for c in cases], [2], f_last[b], base.vis_start[b], base.vis_len[b], 0.1, SCALE, acc64=True)
            for l in range(L):
                _check_out(out[l, b], tr.outputs[l])
            assert fix[b, :ks[b]].cpu().tolist() == tr.f_last.tolist()
            f_last[b] = tr.f_last
    assert ctx.device_faults() == 0


def _head_shard(cases, r, world):
    """Rank r's share of a layer stack: its KV heads (and the query heads that read them) of every layer."""
    from harness import Case
    import paper_2605_17447_b200 as f
    base = cases[0]
    q0, q1, k0, k1 = f.shard_heads(base.H, base.Hkv, r, world)
    local, views, shared = [], [], None
    for c in cases:
        lc = Case(c.B, q1 - q0, k1 - k0, c.seq_len, c.vis_start, c.vis_len, c.K[:, :, k0:k1].contiguous(),
                  c.V[:, :, k0:k1].contiguous(), c.q[:, q0:q1].contiguous(), c.page_size, c.block_table, c.num_pages)
        v = lc.device_view()
        if shared is None:
            shared = (v.seq_len, v.vis_start, v.vis_len)
        views.append(f.KVView(v.k, v.v, shared[0], shared[1], shared[2], q1 - q0, max(c.seq_len), SCALE,
                              block_table=v.block_table if c.page_size else None))
        local.append(lc)
    return local, views, torch.stack([c.q for c in local]), (q0, q1)


@pytest.mark.parametrize("paged", [False, True])
def test_decode_step_with_heads_sharded_over_two_ranks(fo, paged):
    """Heads sharded over two processes, emulated one rank after the other on one GPU: each rank runs the
    whole step over its 14 query / 2 KV heads, and at every focal layer its exchange callback adds the other
    rank's local scores (what the all-reduce would deliver) before the selection. Both ranks must select
    the oracle's all-head sets and produce the oracle's outputs for their heads."""
    L, world = 5, 2
    spans = [(6, 300, 20), (3, 170, 41), (9, 512, 7)]
    focal = [1, 3]
    cases, _, _ = make_layer_stack(2500, spans, L, page_size=16 if paged else 0, q_boost=1.5)
    base = cases[0]
    ks = [oracle.kept_count(n, 0.1) for n in base.vis_len]
    n_max = max(base.vis_len)
    ranks = []
    for r in range(world):
        local, views, q_all, (q0, q1) = _head_shard(cases, r, world)
        c = fo.Context(max_batch=base.B, num_q_heads=q1 - q0, num_kv_heads=base.Hkv // world, max_seq_len=max(base.seq_len),
                       max_vis_len=n_max + 13)
        # what this rank would contribute to the exchange at each layer: the mean over its heads
        part = torch.zeros(L, base.B, n_max, dtype=torch.float32, device="cuda")
        scratch = torch.empty(base.B, q1 - q0, 128, dtype=torch.float32, device="cuda")
        for l in range(L):
            fo.fastocr_dense_decode_attn(c, views[l], q_all[l].cuda(), scratch, scores_out=part[l])
        ranks.append(dict(ctx=c, views=views, q=q_all.cuda(), heads=(q0, q1), part=part,
                          fix=torch.full((base.B, max(ks)), -1, dtype=torch.int32, device="cuda"), have=False, calls=[]))
    kd = torch.tensor(ks, dtype=torch.int32, device="cuda")
    f_last = [None] * base.B
    for step in range(2):
        traces = [oracle.decode_step([c.seq(b) for c in cases], focal, f_last[b], base.vis_start[b], base.vis_len[b], 0.1, SCALE,
                                     acc64=True) for b in range(base.B)]
        for r, me in enumerate(ranks):
            other = ranks[1 - r]

            def exchange(scores, layer, me=me, other=other):
                assert scores.shape == (base.B, n_max + 13) and scores.dtype == torch.float32 and scores.is_cuda
                me["calls"].append(layer)
                # the library's local scores are what the stand-alone call gave for this rank
                for b in range(base.B):
                    assert torch.equal(scores[b, :base.vis_len[b]], me["part"][layer, b, :base.vis_len[b]])
                scores[:, :n_max] += other["part"][layer]

            out = torch.full((L, base.B, me["heads"][1] - me["heads"][0], 128), 7.0, dtype=torch.float32, device="cuda")
            me["have"] = fo.fastocr_decode_step(me["ctx"], me["views"], me["q"], out, [l in focal for l in range(L)], kd, me["fix"],
                                                me["have"], n_max, scores_exchange=exchange)
            assert me["have"]
            for b in range(base.B):
                for l in range(L):
                    _check_out(out[l, b], traces[b].outputs[l][me["heads"][0]:me["heads"][1]])
                assert me["fix"][b, :ks[b]].cpu().tolist() == traces[b].f_last.tolist()
            assert me["ctx"].device_faults() == 0
        assert torch.equal(ranks[0]["fix"], ranks[1]["fix"])
        for b in range(base.B):
            f_last[b] = traces[b].f_last
    # one exchange per focal layer, in layer order; the first step's fallback at layer 0 included
    assert ranks[0]["calls"] == [0, 1, 3, 1, 3] and ranks[1]["calls"] == ranks[0]["calls"]
    for me in ranks:
        me["ctx"].close()


def test_a_failing_scores_exchange_ends_the_step(fo, ctx):
    """What the exchange callable raises reaches the caller, and nothing is selected after it."""
    L = 3
    cases, views, q_all = make_layer_stack(2600, [(4, 200, 10)], L)
    base = cases[0]
    kd = torch.tensor([20], dtype=torch.int32, device="cuda")
    fix = torch.full((1, 20), -1, dtype=torch.int32, device="cuda")
    out = torch.empty(L, 1, 28, 128, dtype=torch.float32, device="cuda")

    def boom(scores, layer):
        raise RuntimeError("exchange failed on purpose (host side)")

    with pytest.raises(RuntimeError, match="exchange failed on purpose"):
        fo.fastocr_decode_step(ctx, views, q_all.cuda(), out, [False, True, False], kd, fix, False, base.vis_len[0], scores_exchange=boom)
    torch.cuda.synchronize()
    assert fix.cpu().tolist() == [[-1] * 20]
    # the context is usable afterwards
    assert fo.fastocr_decode_step(ctx, views, q_all.cuda(), out, [False, True, False], kd, fix, False, base.vis_len[0])
    tr = oracle.decode_step([c.seq(0) for c in cases], [1], None, base.vis_start[0], base.vis_len[0], 0.1, SCALE, acc64=True)
    assert fix[0].cpu().tolist() == tr.f_last.tolist()


_NCCL_WORKER = r"""
import os, sys, torch, torch.distributed as dist
root = os.environ["FASTOCR_ROOT"]
sys.path.insert(0, root); sys.path.insert(0, os.path.join(root, "tests"))
import oracle
import paper_2605_17447_b200 as fo
from harness import SCALE, make_layer_stack
torch.cuda.set_device(0)
dist.init_process_group("nccl", init_method="tcp://127.0.0.1:%s" % os.environ["PORT"], rank=0, world_size=1)
warm = torch.ones(4, device="cuda"); dist.all_reduce(warm); torch.cuda.synchronize()
print("backend up", flush=True)
L, spans, focal = 4, [(6, 300, 20), (3, 170, 41)], [2]
cases, views, q_all = make_layer_stack(2700, spans, L, q_boost=1.5)
base = cases[0]
ks = [oracle.kept_count(n, 0.1) for n in base.vis_len]
kd = torch.tensor(ks, dtype=torch.int32, device="cuda")
fix = torch.full((base.B, max(ks)), -1, dtype=torch.int32, device="cuda")
ctx = fo.Context(max_batch=base.B, num_q_heads=28, num_kv_heads=4, max_seq_len=max(base.seq_len), max_vis_len=max(base.vis_len))
out = torch.empty(L, base.B, 28, 128, dtype=torch.float32, device="cuda")
have, f_last = False, [None] * base.B
for step in range(2):
    have = fo.fastocr_decode_step(ctx, views, q_all.cuda(), out, [l in focal for l in range(L)], kd, fix, have, max(base.vis_len),
                                  scores_exchange=fo.make_scores_exchange())
    torch.cuda.synchronize()
    for b in range(base.B):
        tr = oracle.decode_step([c.seq(b) for c in cases], focal, f_last[b], base.vis_start[b], base.vis_len[b], 0.1, SCALE, acc64=True)
        for l in range(L):
            assert float((out[l, b].cpu() - tr.outputs[l]).abs().max()) <= 1e-4
        assert fix[b, :ks[b]].cpu().tolist() == tr.f_last.tolist()
        f_last[b] = tr.f_last
ratio = torch.tensor([[0.25, 0.5]], device="cuda")
assert fo.mean_ratio_over_ranks(ratio).cpu().tolist() == [[0.25, 0.5]]
assert ctx.device_faults() == 0
ctx.close()
dist.destroy_process_group()
print("ok")
"""


def test_scores_exchange_over_nccl_single_rank(tmp_path):
    """The exchange helper as a user would pass it, over the NCCL backend (one rank: the only size one GPU
    allows): the library's score workspace reaches torch.distributed as a tensor, the collective is ordered
    between the library's launches on the current stream, and the step matches the oracle."""
    import os
    import socket
    import subprocess
    import sys
    s = socket.socket(); s.bind(("127.0.0.1", 0)); port = s.getsockname()[1]; s.close()
    script = tmp_path / "n.py"
    script.write_text(_NCCL_WORKER)
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    env = dict(os.environ, PORT=str(port), FASTOCR_ROOT=root, NCCL_NVLS_ENABLE="0")
    p = subprocess.run([sys.executable, str(script)], env=env, capture_output=True, text=True, timeout=300)
    if "backend up" not in p.stdout:                    # the machine's NCCL set-up, not this library
        pytest.skip("the NCCL backend did not come up here: " + p.stderr[-300:])
    assert p.returncode == 0 and p.stdout.strip().endswith("ok"), p.stdout[-2000:] + p.stderr[-4000:]


@pytest.mark.parametrize("paged", [False, True])
def test_batches_beyond_one_launch_run_in_chunks(fo, paged):
    """140 sequences x 4 KV heads = 560 (sequence, KV head) pairs, more than a launch covers (512): every entry
    point processes the batch as chunks of whole sequences (128 + 12 here). Every sequence is compared with the
    oracle: single-layer calls, the warm-up step, and the decode step with per-sequence focal sets (so that the
    focal matrix, the index rows and the outputs are all addressed per chunk), plain and as the union variant."""
    g = torch.Generator().manual_seed(91)
    B, L = 140, 4
    spans = [(int(torch.randint(0, 7, (1,), generator=g)), int(torch.randint(40, 121, (1,), generator=g)),
              int(torch.randint(0, 21, (1,), generator=g))) for _ in range(B)]
    cases, views, q_all = make_layer_stack(2800, spans, L, page_size=16 if paged else 0, q_boost=1.5)
    base = cases[0]
    n_max = max(base.vis_len)
    c = fo.Context(max_batch=B, num_q_heads=28, num_kv_heads=4, max_seq_len=max(base.seq_len), max_vis_len=n_max)
    ks = [oracle.kept_count(n, 0.1) for n in base.vis_len]
    kd = torch.tensor(ks, dtype=torch.int32, device="cuda")
    qd = q_all.cuda()

    # single-layer entry points
    out = torch.empty(B, 28, 128, dtype=torch.float32, device="cuda")
    sc = torch.zeros(B, n_max, dtype=torch.float32, device="cuda")
    mass = torch.zeros(B, dtype=torch.float32, device="cuda")
    fo.fastocr_dense_decode_attn(c, views[0], qd[0], out, scores_out=sc, image_mass_out=mass)
    sc2 = torch.zeros_like(sc)
    fo.fastocr_focal_scores(c, views[0], qd[0], sc2)
    idx = torch.full((B, max(ks)), -1, dtype=torch.int32, device="cuda")
    fo.fastocr_select_topk(c, sc, views[0].vis_len, kd, idx, n_max)
    out_s = torch.empty_like(out)
    fo.fastocr_sparse_decode_attn(c, views[0], qd[0], idx, kd, out_s)
    assert torch.equal(sc, sc2)
    for b in range(B):
        qb, Kb, Vb = cases[0].seq(b)
        _check_out(out[b], oracle.dense(qb, Kb, Vb, SCALE, True))
        ref_sc, ref_mass = oracle.scores(qb, Kb, SCALE, base.vis_start[b], base.vis_len[b], True)
        assert float((sc[b, :base.vis_len[b]].cpu() - ref_sc).abs().max()) <= 1e-6
        assert abs(float(mass[b]) - ref_mass) <= 1e-5
        want = oracle.topk(sc[b, :base.vis_len[b]].cpu(), ks[b])
        assert idx[b, :ks[b]].cpu().tolist() == want.tolist()
        _check_out(out_s[b], oracle.sparse(qb, Kb, Vb, SCALE, base.vis_start[b], base.vis_len[b], want, True))

    # warm-up step: Eq. 1's ratio per layer and sequence
    outw = torch.empty(L, B, 28, 128, dtype=torch.float32, device="cuda")
    r = torch.full((L, B), -1.0, dtype=torch.float32, device="cuda")
    fo.fastocr_warmup_step(c, views, qd, outw, r)
    for b in (0, 1, 126, 127, 128, 129, 139):           # both sides of the chunk boundary
        outs, rr = oracle.warmup_step([cs.seq(b) for cs in cases], base.vis_start[b], base.vis_len[b], SCALE, acc64=True)
        for l in range(L):
            _check_out(outw[l, b], outs[l])
            assert abs(float(r[l, b]) - rr[l]) <= 1e-5

    # decode steps with per-sequence focal layer sets
    focal_of = [[1] if b % 3 == 0 else ([2] if b % 3 == 1 else [1, 3]) for b in range(B)]
    matrix = [[l in focal_of[b] for b in range(B)] for l in range(L)]
    for union in (False, True):
        fix = torch.full((B, max(ks)), -1, dtype=torch.int32, device="cuda")
        have, f_last = False, [None] * B
        for step in range(2):
            outd = torch.full((L, B, 28, 128), 7.0, dtype=torch.float32, device="cuda")
            have = fo.fastocr_decode_step(c, views, qd, outd, matrix, kd, fix, have, n_max, union_sets=union,
                                          max_kept=max(3 * k + s - n for k, s, n in zip(ks, base.seq_len, base.vis_len)) if union else 0)
            assert have
            for b in range(B):
                tr = oracle.decode_step([cs.seq(b) for cs in cases], focal_of[b], f_last[b], base.vis_start[b], base.vis_len[b],
                                        0.1, SCALE, acc64=True, union_sets=union)
                for l in range(L):
                    _check_out(outd[l, b], tr.outputs[l])
                assert fix[b, :ks[b]].cpu().tolist() == tr.f_last.tolist()
                f_last[b] = tr.f_last
    assert c.device_faults() == 0
    c.close()


def test_two_contexts_on_two_streams_and_a_captured_step(fo):
    """Launches go to the stream they are given: two contexts, each on a stream of its own, run their steps
    at the same time on different data; then one step is captured into a CUDA graph and replayed on fresh
    queries (the pointers are the same, the contents new). All of it against the oracle."""
    L, focal = 4, [1]
    spans = [(6, 300, 20), (3, 170, 41)]
    jobs = []
    for seed in (2900, 2901):
        cases, views, q_all = make_layer_stack(seed, spans, L, q_boost=1.5)
        base = cases[0]
        ks = [oracle.kept_count(n, 0.1) for n in base.vis_len]
        jobs.append(dict(cases=cases, views=views, q=q_all.cuda(), base=base, ks=ks,
                         ctx=fo.Context(max_batch=base.B, num_q_heads=28, num_kv_heads=4, max_seq_len=max(base.seq_len),
                                        max_vis_len=max(base.vis_len)),
                         kd=torch.tensor(ks, dtype=torch.int32, device="cuda"),
                         fix=torch.full((base.B, max(ks)), -1, dtype=torch.int32, device="cuda"),
                         out=torch.full((L, base.B, 28, 128), 7.0, dtype=torch.float32, device="cuda"),
                         stream=torch.cuda.Stream()))
    torch.cuda.synchronize()
    for rep in range(3):                                 # interleaved issue: the two streams overlap on the device
        for j in jobs:
            fo.fastocr_decode_step(j["ctx"], j["views"], j["q"], j["out"], [l in focal for l in range(L)], j["kd"], j["fix"],
                                   rep > 0, max(j["base"].vis_len), stream=j["stream"])
    torch.cuda.synchronize()
    for j in jobs:
        base = j["base"]
        for b in range(base.B):
            tr = oracle.decode_step([c.seq(b) for c in j["cases"]], focal, None, base.vis_start[b], base.vis_len[b], 0.1, SCALE, acc64=True)
            tr2 = oracle.decode_step([c.seq(b) for c in j["cases"]], focal, tr.f_last, base.vis_start[b], base.vis_len[b], 0.1, SCALE, acc64=True)
            for l in range(L):
                _check_out(j["out"][l, b], tr2.outputs[l])
            assert j["fix"][b, :j["ks"][b]].cpu().tolist() == tr2.f_last.tolist()
            j.setdefault("f_last", []).append(tr2.f_last)

    # capture one step of the first job, replay it on new queries written into the same buffer
    j = jobs[0]
    g = torch.cuda.CUDAGraph()
    side = torch.cuda.Stream()
    with torch.cuda.graph(g, stream=side):
        fo.fastocr_decode_step(j["ctx"], j["views"], j["q"], j["out"], [l in focal for l in range(L)], j["kd"], j["fix"], True,
                               max(j["base"].vis_len))                  # the current stream is the capturing one
    cases2, _, q2 = make_layer_stack(2900, spans, L, q_boost=1.1)       # same caches (same seed), other queries
    j["q"].copy_(q2.cuda())
    j["out"].fill_(7.0)
    g.replay()
    torch.cuda.synchronize()
    base = j["base"]
    for b in range(base.B):
        tr = oracle.decode_step([c.seq(b) for c in cases2], focal, j["f_last"][b], base.vis_start[b], base.vis_len[b], 0.1, SCALE, acc64=True)
        for l in range(L):
            _check_out(j["out"][l, b], tr.outputs[l])
        assert j["fix"][b, :j["ks"][b]].cpu().tolist() == tr.f_last.tolist()
    for j in jobs:
        assert j["ctx"].device_faults() == 0
        j["ctx"].close()


def _random_step_case(seed):
    """One seeded random decode-step problem: head geometry, batch, depth, spans (empty image, empty text,
    single tokens, ragged), cache layout, tau, focal sets (one per batch or per sequence), plain or union."""
    import random
    rnd = random.Random(seed)
    H, Hkv = rnd.choice([(28, 4), (16, 2), (12, 2), (8, 8), (64, 8), (10, 2), (6, 2), (4, 1), (7, 1), (32, 4)])
    B, L = rnd.choice([1, 2, 3, 5, 9]), rnd.choice([1, 2, 3, 5, 7])
    paged, big = rnd.random() < 0.5, rnd.random() < 0.15
    tau = rnd.choice([0.0, 0.004, 0.05, 0.1, 0.3, 1.0])
    spans = []
    for _ in range(B):
        n = rnd.choice([3000, 5000]) if big else rnd.choice([0, 1, 7, 33, 64, 100, 257, 700, 1500])
        a, t = rnd.choice([0, 1, 5, 16, 40]), rnd.choice([0, 1, 3, 20, 70, 200])
        if a + t == 0 and oracle.kept_count(n, tau) == 0:
            a = 1                                        # the oracle refuses an empty kept set
        spans.append((a, n, t))
    if rnd.random() < 0.4:
        focal_of = [[l for l in range(L) if rnd.random() < 0.35] for _ in range(B)]
        is_focal = [[l in focal_of[b] for b in range(B)] for l in range(L)]
    else:
        f = [l for l in range(L) if rnd.random() < 0.35]
        focal_of, is_focal = [f] * B, [l in f for l in range(L)]
    return dict(H=H, Hkv=Hkv, L=L, paged=paged, tau=tau, spans=spans, focal_of=focal_of, is_focal=is_focal,
                union=rnd.random() < 0.3, steps=rnd.choice([1, 2, 3]), boost=rnd.choice([1.0, 1.5, 2.5]))


@pytest.mark.parametrize("block", range(4))
def test_randomised_decode_steps(fo, block):
    """Forty seeded random decode-step problems (ten per block), each run for one to three steps and
    compared with the oracle's Algorithm 1 trace: every output, and the carried set exactly."""
    for seed in range(10 * block, 10 * block + 10):
        p = _random_step_case(seed)
        cases, views, q_all = make_layer_stack(100000 + seed, p["spans"], p["L"], H=p["H"], Hkv=p["Hkv"],
                                               page_size=16 if p["paged"] else 0, q_boost=p["boost"])
        base = cases[0]
        B, L = base.B, p["L"]
        ks = [oracle.kept_count(n, p["tau"]) for n in base.vis_len]
        kd = torch.tensor(ks, dtype=torch.int32, device="cuda")
        fix = torch.full((B, max(1, max(ks))), -1, dtype=torch.int32, device="cuda")
        n_max = max(1, max(base.vis_len))
        c = fo.Context(max_batch=B, num_q_heads=p["H"], num_kv_heads=p["Hkv"], max_seq_len=max(base.seq_len), max_vis_len=n_max)
        have, f_last = False, [None] * B
        for step in range(p["steps"]):
            out = torch.full((L, B, p["H"], 128), 7.0, dtype=torch.float32, device="cuda")
            mk = max(L * k + s - n for k, s, n in zip(ks, base.seq_len, base.vis_len)) if p["union"] else 0
            have = fo.fastocr_decode_step(c, views, q_all.cuda(), out, p["is_focal"], kd, fix, have, n_max, max_kept=mk, union_sets=p["union"])
            for b in range(B):
                tr = oracle.decode_step([cs.seq(b) for cs in cases], p["focal_of"][b], f_last[b], base.vis_start[b], base.vis_len[b],
                                        p["tau"], SCALE, acc64=True, union_sets=p["union"])
                for l in range(L):
                    err = float((out[l, b].cpu() - tr.outputs[l]).abs().max())
                    assert err <= TIGHT, (seed, step, l, b, err, p)
                if tr.f_last is not None:
                    assert fix[b, :ks[b]].cpu().tolist() == tr.f_last.tolist(), (seed, step, b, p)
                f_last[b] = tr.f_last
        assert c.device_faults() == 0, (seed, p)
        c.close()

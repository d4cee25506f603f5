"""Parity at the benchmark's full size and launch configuration (batch 64, N = 8192, 7B-shaped
heads, contiguous cache): sampled sequences are checked one by one against the oracle; properties
that hold at any size are checked on the whole batch."""
import math

import numpy as np
import pytest
import torch

import oracle

pytestmark = pytest.mark.gpu
SCALE = 1.0 / math.sqrt(128.0)


def test_full_size_layer_chain_against_oracle_on_sampled_sequences():
    import paper_2605_17447_b200 as fo
    from workloads import fixation_track, get_config, make_kv, make_queries
    cfg = get_config("cfg4", N=8192, batch=64)
    dev = "cuda"
    B, H, Hkv, N = cfg.batch, cfg.num_q_heads, cfg.num_kv_heads, cfg.vis_len[0]
    S = cfg.seq_len(0)[0] + 1
    K, V = make_kv(cfg.seed, 0, B, S, Hkv, 128, dev)
    centres = torch.tensor(np.array([fixation_track(cfg.seed, b, 1, cfg.grid_h[b], cfg.grid_w[b], cfg.advance)[0] for b in range(B)]), device=dev)
    i32 = lambda x: torch.tensor(x, dtype=torch.int32, device=dev)
    vs = i32(cfg.vis_start)
    q = make_queries(cfg.seed, 0, 0, lambda b, pos: K[b, pos], vs.long(), centres,
                     torch.tensor(cfg.grid_h, device=dev), torch.tensor(cfg.grid_w, device=dev), H)
    k = fo.kept_count(N, cfg.tau)
    assert k == 410
    ctx = fo.Context(B, H, Hkv, S, N)
    kv = fo.KVView(K, V, i32([S] * B), vs, i32(cfg.vis_len), H, S, SCALE)
    dense = torch.empty(B, H, 128, dtype=torch.float32, device=dev)
    out = torch.empty_like(dense)
    sc = torch.zeros(B, N, dtype=torch.float32, device=dev)
    idx = torch.zeros(B, k, dtype=torch.int32, device=dev)
    kd = i32([k] * B)
    fo.fastocr_dense_decode_attn(ctx, kv, q, dense, scores_out=sc)
    fo.fastocr_select_topk(ctx, sc, kv.vis_len, kd, idx, N)
    fo.fastocr_sparse_decode_attn(ctx, kv, q, idx, kd, out)
    torch.cuda.synchronize()
    assert ctx.device_faults() == 0
    # whole batch: selections are ascending, distinct, in range, and are the top-k of the GPU's own scores
    assert bool((idx[:, 1:] > idx[:, :-1]).all()) and int(idx.min()) >= 0 and int(idx.max()) < N
    kth = torch.gather(sc, 1, idx.long()).min(dim=1).values
    assert bool(((sc > kth[:, None]).sum(dim=1) < k).all())
    # image mass of Eq. 1 lies in (0, 1)
    mass = sc.sum(dim=1)
    assert bool((mass > 0).all()) and bool((mass < 1).all())
    # tau = 1 through the pruned path reproduces the dense output
    full = torch.arange(N, dtype=torch.int32, device=dev).repeat(B, 1).contiguous()
    out_full = torch.empty_like(dense)
    fo.fastocr_sparse_decode_attn(ctx, kv, q, full, i32([N] * B), out_full)
    assert float((out_full - dense).abs().max()) <= 1e-5
    # the decode step (scores formed inside the selection kernel, a cluster of CTAs per sequence,
    # launches overlapping) gives the same bits as the separate calls
    fix = torch.full((B, k), -1, dtype=torch.int32, device=dev)
    out2 = torch.empty(3, B, H, 128, dtype=torch.float32, device=dev)    # two pruned layers: they run from a launch plan
    have = fo.fastocr_decode_step(ctx, [kv, kv, kv], torch.stack([q, q, q]), out2, [True, False, False], kd, fix, False, N)
    torch.cuda.synchronize()
    assert have and torch.equal(fix, idx)
    assert torch.equal(out2[0], dense) and torch.equal(out2[1], out) and torch.equal(out2[2], out)
    # sampled sequences against the oracle, element by element
    for b in (0, 17, 63):
        qc, Kc, Vc = q[b].cpu(), K[b].cpu(), V[b].cpu()
        ref_sc, _ = oracle.scores(qc, Kc, SCALE, cfg.vis_start[b], N, True)
        assert bool(((sc[b].cpu() - ref_sc).abs() <= 2e-5 * ref_sc + 1e-12).all())
        sel = idx[b].cpu()
        assert sel.tolist() == oracle.topk(sc[b].cpu(), k).tolist()
        ref_idx = oracle.topk(ref_sc, k)
        diff = set(sel.tolist()) ^ set(ref_idx.tolist())
        kth_ref = float(torch.sort(ref_sc, descending=True).values[k - 1])
        assert all(abs(float(ref_sc[i]) - kth_ref) <= 1e-5 * kth_ref for i in diff)
        for got, ref in ((dense[b], oracle.dense(qc, Kc, Vc, SCALE, True)),
                         (out[b], oracle.sparse(qc, Kc, Vc, SCALE, cfg.vis_start[b], N, sel, True))):
            err = (got.cpu() - ref).abs()
            assert err.max() <= 1e-4 and err.mean() <= 1e-3
    ctx.close()

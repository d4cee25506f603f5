"""No-GPU checks: the built library loads, exports every symbol the header declares, and its
host-only entry points agree with the oracle's rules; sequence sharding over gloo ranks."""
import os
import re
import subprocess
import sys

import pytest

import oracle

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_library_exports_every_declared_symbol():
    from paper_2605_17447_b200 import _lib, build
    build.build()
    header = open(os.path.join(ROOT, "include", "fastocr.h")).read()
    declared = set(re.findall(r"\b(fastocr_[a-z_]+)\s*\(", header))
    assert {"fastocr_focal_scores", "fastocr_select_topk", "fastocr_sparse_decode_attn",
            "fastocr_dense_decode_attn", "fastocr_decode_step"} <= declared
    lib = _lib.load()
    for name in declared:
        assert hasattr(lib, name), name
    assert declared == set(_lib.EXPORTS), declared ^ set(_lib.EXPORTS)


def test_host_rules_agree_with_oracle():
    import paper_2605_17447_b200 as fo
    for n in (0, 1, 20, 77, 1000, 1024, 4096, 8192, 16384, 32768):
        for tau in (0.0, 0.004, 0.02, 0.05, 0.1, 0.2, 0.25, 1.0, 1.5):
            assert fo.kept_count(n, tau) == oracle.kept_count(n, tau), (n, tau)
    import random
    rnd = random.Random(4)
    for _ in range(200):
        L = rnd.randint(1, 40)
        r = [rnd.choice([0.1, 0.2, 0.3, rnd.random()]) for _ in range(L)]
        rho, gap = rnd.choice([0.05, 0.1, 0.2, 0.5, 1.0]), rnd.randint(0, 4)
        assert fo.focal_layers(r, rho, gap) == oracle.focal_layers(r, rho, gap)
    assert abs(fo.attn_flops(8, 36, 2048, 4096) - oracle.attn_flops(8, 36, 2048, 4096)) < 1.0
    for b, l, h, s_, f, sk in ((8, 36, 2048, 4096, 4, 204.8), (4, 36, 2048, 8192, 3, 409.6), (64, 28, 3584, 8449, 2, 666), (1, 5, 64, 100, 0, 0)):
        want = oracle.attn_flops_pruned(b, l, h, s_, f, sk)
        assert abs(fo.attn_flops_pruned(b, l, h, s_, f, sk) - want) <= 1e-9 * want


def test_product_does_not_import_the_oracle():
    pkg = os.path.join(ROOT, "paper_2605_17447_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".h", ".cuh")):
                assert "oracle" not in open(os.path.join(dirpath, f)).read().lower().replace("no cpu or pytorch", ""), f


_GLOO_WORKER = r"""
import os, sys, torch, torch.distributed as dist
sys.path.insert(0, os.environ["FASTOCR_ROOT"])
from paper_2605_17447_b200.sharding import shard_sequences
dist.init_process_group("gloo", init_method="tcp://127.0.0.1:%s" % os.environ["PORT"],
                        rank=int(os.environ["RANK"]), world_size=int(os.environ["WORLD_SIZE"]))
B = 33
lo, hi = shard_sequences(B, dist.get_rank(), dist.get_world_size())
own = torch.zeros(B, dtype=torch.int64); own[lo:hi] = 1
units = torch.tensor([float(hi - lo)]); t = torch.tensor([1.0 + dist.get_rank()])
dist.all_reduce(own); dist.all_reduce(units); dist.all_reduce(t, op=dist.ReduceOp.MAX)
assert own.tolist() == [1] * B, own          # every sequence owned exactly once
assert units.item() == B and t.item() == dist.get_world_size()
dist.barrier(); dist.destroy_process_group()
"""


def test_sequence_sharding_world_size_two_gloo(tmp_path):
    import socket
    s = socket.socket(); s.bind(("127.0.0.1", 0)); port = s.getsockname()[1]; s.close()
    script = tmp_path / "w.py"
    script.write_text(_GLOO_WORKER)
    procs = []
    for r in range(2):
        env = dict(os.environ, RANK=str(r), WORLD_SIZE="2", PORT=str(port), FASTOCR_ROOT=ROOT)
        procs.append(subprocess.Popen([sys.executable, str(script)], env=env))
    for p in procs:
        assert p.wait(timeout=120) == 0


def test_shard_sequences_edges():
    from paper_2605_17447_b200.sharding import shard_sequences
    assert [shard_sequences(5, r, 8) for r in range(8)] == [(0, 1), (1, 2), (2, 3), (3, 4), (4, 5), (5, 5), (5, 5), (5, 5)]
    assert shard_sequences(64, 3, 8) == (24, 32)
    with pytest.raises(ValueError):
        shard_sequences(4, 2, 2)


_GLOO_HEADS_WORKER = r"""
import os, sys, math, torch, torch.distributed as dist
sys.path.insert(0, os.environ["FASTOCR_ROOT"])
import oracle
from paper_2605_17447_b200.sharding import shard_heads, make_scores_exchange, mean_ratio_over_ranks
dist.init_process_group("gloo", init_method="tcp://127.0.0.1:%s" % os.environ["PORT"],
                        rank=int(os.environ["RANK"]), world_size=int(os.environ["WORLD_SIZE"]))
rank, world = dist.get_rank(), dist.get_world_size()
# one sequence, 8 query heads over 4 KV heads; the same seeded tensors on every rank
H, Hkv, d, vs, N, T = 8, 4, 128, 5, 300, 40
S = vs + N + T
g = torch.Generator().manual_seed(77)
K = torch.randn(S, Hkv, d, generator=g).bfloat16()
q = (torch.randn(H, d, generator=g) * 1.5).bfloat16()
sm = 1 / math.sqrt(d)
want_scores, want_mass = oracle.scores(q, K, sm, vs, N)            # all heads
q0, q1, k0, k1 = shard_heads(H, Hkv, rank, world)
assert (q1 - q0) * world == H and (k1 - k0) * world == Hkv
local, mass = oracle.scores(q[q0:q1], K[:, k0:k1].contiguous(), sm, vs, N)   # this rank's heads only
summed = local.clone().view(1, N)
make_scores_exchange()(summed, 0)                                   # the product's exchange, over gloo
# the sum of the local means is world x the mean over all heads (up to rounding): same ranking
assert torch.allclose(summed[0] / world, want_scores, rtol=2e-6, atol=1e-9), (summed[0] / world - want_scores).abs().max()
k = 15
got, want = set(oracle.topk(summed[0], k).tolist()), set(oracle.topk(want_scores, k).tolist())
if got != want:                                                     # only tokens tied with the k-th score to rounding may differ
    kth = torch.sort(want_scores, descending=True).values[k - 1].item()
    for i in got ^ want:
        assert abs(want_scores[i].item() - kth) <= 1e-5 * abs(kth), (i, want_scores[i].item(), kth)
# every rank ends with the same bits, hence the same selection
mine = summed.clone(); other = [torch.empty_like(mine) for _ in range(world)]
dist.all_gather(other, mine)
assert all(torch.equal(o, mine) for o in other)
r = mean_ratio_over_ranks(torch.tensor([[mass]], dtype=torch.float32))
assert abs(r.item() - want_mass) <= 1e-5
dist.barrier(); dist.destroy_process_group()
"""


def test_head_sharding_world_size_two_gloo(tmp_path):
    """Heads sharded over two ranks: the exchanged local score means select what the all-head scores
    select (Section 3.1.1 averages over all heads), identically on both ranks."""
    import socket
    s = socket.socket(); s.bind(("127.0.0.1", 0)); port = s.getsockname()[1]; s.close()
    script = tmp_path / "h.py"
    script.write_text(_GLOO_HEADS_WORKER)
    procs = []
    for r in range(2):
        env = dict(os.environ, RANK=str(r), WORLD_SIZE="2", PORT=str(port), FASTOCR_ROOT=ROOT)
        procs.append(subprocess.Popen([sys.executable, str(script)], env=env))
    for p in procs:
        assert p.wait(timeout=180) == 0


def test_shard_heads_edges():
    from paper_2605_17447_b200.sharding import shard_heads
    assert [shard_heads(64, 8, r, 4) for r in range(4)] == [(0, 16, 0, 2), (16, 32, 2, 4), (32, 48, 4, 6), (48, 64, 6, 8)]
    assert shard_heads(28, 4, 0, 1) == (0, 28, 0, 4)
    with pytest.raises(ValueError):
        shard_heads(28, 4, 0, 3)        # 4 KV heads do not divide over 3 ranks
    with pytest.raises(ValueError):
        shard_heads(30, 4, 0, 2)
